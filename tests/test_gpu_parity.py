"""CUDA path vs fp64 oracle through the C ABI, element by element, on seeded inputs small enough for the
oracle to finish in seconds but spanning several tiles, ragged tails and the degenerate cases."""
import numpy as np
import pytest
import torch

from oracle import fi_oracle as fo
from paper_2002_02645_b200 import binding as fb
from paper_2002_02645_b200 import datagen as dg
from helpers import compare_cascade, compare_lookup, f32, make_cache, tau_between, to_device

pytestmark = pytest.mark.gpu


def run_lookup(cache, queries_np, **kw):
    q = to_device(queries_np, cache.device)
    out = cache.lookup_batch(q, **kw)
    torch.cuda.synchronize()
    cache.poll_status()
    return (out.label.cpu().numpy(), out.conf.cpu().numpy(), out.hit.cpu().numpy(), out.topk_dist.cpu().numpy(),
            out.topk_idx.cpu().numpy())


def check_case(stage, *, k, num_classes, rule, path, percentile=50.0, metric=0, weights=None, twice=True):
    storage = stage.dtype
    ref0 = fo.lookup(stage.queries, stage.cache_vecs, stage.cache_labels, k=k, tau=0.0, rule=rule, metric=metric,
                     weights=weights)
    if rule == fo.RULE_CONF_GT:
        tau = tau_between(ref0.conf, percentile)
    else:
        near = np.sqrt(ref0.nd[:, 0]) if metric == 1 else ref0.nd[:, 0]
        tau = tau_between(near, percentile)
    ref = fo.lookup(stage.queries, stage.cache_vecs, stage.cache_labels, k=k, tau=tau, rule=rule, metric=metric,
                    weights=weights)
    cache = make_cache(stage, k=k, num_classes=num_classes, rule=rule, metric=metric, tau=tau,
                       max_batch=max(stage.queries.shape[0], 1), path=path, weights=weights)
    got = run_lookup(cache, stage.queries)
    stats = compare_lookup(*got, ref, storage=storage, tau=tau, rule=rule, metric=metric,
                           cache_labels=stage.cache_labels, weights=weights)
    if twice:   # a race would show as run-to-run differences
        again = run_lookup(cache, stage.queries)
        for a, b in zip(got, again):
            np.testing.assert_array_equal(a, b)
    print(stats)
    assert stats.exempt_gap <= max(2, stage.queries.shape[0] // 5)
    assert 0 < ref.hit.sum() < ref.hit.shape[0] or stage.queries.shape[0] < 4
    cache.close()
    return stats


# ------------------------------------------------------------------ config 1: fp32, k = 1, exact copies, DIST_LE

def test_config1_full():
    w = dg.config1(seed=0)
    st = w.stages[0]
    x64 = st.cache_vecs.astype(np.float64)
    # 20th percentile of squared distances between distinct cache entries of equal label
    d = []
    for c in range(10):
        xc = x64[st.cache_labels == c]
        D = ((xc[:, None, :] - xc[None, :, :]) ** 2).sum(-1)
        d.append(D[np.triu_indices(xc.shape[0], 1)])
    tau = f32(np.percentile(np.concatenate(d), 20.0))
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=1, tau=tau, rule=fo.RULE_DIST_LE)
    cache = make_cache(st, k=1, num_classes=10, rule=fb.FI_HIT_DIST_LE, tau=tau, max_batch=282)
    got = run_lookup(cache, st.queries)
    stats = compare_lookup(*got, ref, storage="f32", tau=tau, rule=1, cache_labels=st.cache_labels)
    print(stats)
    copies = w.meta["copy_of"] >= 0
    assert (got[3][copies, 0] == 0).all() and np.isinf(got[1][copies]).all() and (got[2][copies] == 1).all()
    np.testing.assert_array_equal(got[4][copies, 0], w.meta["copy_of"][copies])
    assert stats.exempt_gap <= 2 and ref.hit.sum() >= 26
    cache.close()


# ------------------------------------------------------------------ streaming path, bf16 and fp32, ragged shapes

@pytest.mark.parametrize("n,d,b,k,dtype", [
    (777, 520, 1, 1, "bf16"), (777, 520, 3, 5, "bf16"), (1501, 64, 4, 10, "bf16"), (333, 2048, 2, 1, "bf16"),
    (9, 8, 4, 5, "bf16"), (1000, 36, 37, 3, "f32"), (257, 4, 5, 32, "f32"), (4100, 16384, 4, 1, "bf16")])
def test_stream_path(n, d, b, k, dtype):
    w = dg.single_layer(name="t", n_cache=n, n_query=b, dim=d, num_classes=7, dtype=dtype, sigma=0.5, k=k, seed=3)
    check_case(w.stages[0], k=k, num_classes=7, rule=fo.RULE_CONF_GT, path=fb.FI_PATH_STREAM)


def test_stream_path_large_dim_reads_queries_in_place():
    # 4 query rows of 65536 bf16 values do not fit in shared memory
    w = dg.single_layer(name="t", n_cache=300, n_query=4, dim=65536, num_classes=5, dtype="bf16", sigma=0.5, k=2, seed=4)
    check_case(w.stages[0], k=2, num_classes=5, rule=fo.RULE_CONF_GT, path=fb.FI_PATH_STREAM)


# ------------------------------------------------------------------ tensor-core path: several tiles, ragged M, N, K

@pytest.mark.parametrize("n,d,b,k", [
    (5003, 200, 300, 5),       # 3 query tiles (last ragged), ragged N, K = 3 blocks + 8
    (40000, 64, 129, 10),      # one k-block, many row ranges, 2 query tiles
    (600, 1024, 5, 1),         # tiny batch, fewer 16-row blocks than CTAs
    (3000, 1024, 2, 5),        # batches of 2 and 3 are copied into a four-row buffer in front of the GEMM
    (700, 4096, 3, 1),
    (16, 8, 17, 5),            # a single 16-row block
    (3000, 4096, 64, 13),      # list length 16, deep K
    (2500, 136, 2200, 29),     # 18 query tiles (two groups), list length 32
    (9990, 4096, 900, 5),      # 4 x 40 tiles of 256 x 256 on 148 SMs: one full tile per CTA plus a tail cut along K
    (12345, 256, 2000, 5),     # short rows, 16 query tiles x 9 long ranges: short first tile, bounds fetched a tile ahead
    (20011, 512, 1100, 10),    # the same with list length 16 (bound slots read on the spot), ragged N and M
    (9000, 320, 2048, 1),      # the same with list length 4, K = 5 blocks
    (33000, 1024, 1100, 5),    # rows of 1,024 values, many entries, batch above 1,024: pairs of CTAs share 256-row tiles
    (40001, 2048, 1024, 10),   # the same with list length 16, ragged entry count, 4 query tiles of a pair exactly
    (9990, 4096, 803, 5),      # deep rows, fewer tiles than CTAs once the last query tile (35 requests) counts half: spans
    (2500, 8192, 190, 5),      # one query tile x 10 cache tiles over 148 CTAs: about 15 pieces per tile
    (7000, 4096, 482, 13),     # two query tiles, list length 16, spans that cross from one tile into the next
    (300, 4096, 200, 29),      # two ragged cache tiles, list length 32, fewer spans than CTAs
])
def test_gemm_path(n, d, b, k):
    w = dg.single_layer(name="t", n_cache=n, n_query=b, dim=d, num_classes=9, dtype="bf16", sigma=0.6, k=k, seed=5)
    check_case(w.stages[0], k=k, num_classes=9, rule=fo.RULE_CONF_GT, path=fb.FI_PATH_GEMM)


@pytest.mark.parametrize("n,d,b,first", [
    (600, 4096, 200, 100),      # spans: three cache tiles, the duplicates inside the first and second
    (9990, 4096, 900, 9500),    # wave + tail: the duplicates sit in tiles that are cut along the row length
    (40000, 256, 300, 7000),    # ranges with the select in the GEMM's epilogue
])
def test_many_equal_scores_keep_the_lowest_indices(n, d, b, first):
    """150 identical cache rows nearer to every query than anything else: every list, queue and merge on the way sees
    150 equal scores and must keep those with the lowest indices, as the oracle's (distance, index) order does."""
    k = 5
    w = dg.single_layer(name="t", n_cache=n, n_query=b, dim=d, num_classes=1, dtype="bf16", sigma=0.6, k=k, seed=11)
    st = w.stages[0]
    # one class: the mean of the queries (rounded to bf16) is nearer to each of them than an independent row is
    mean = torch.from_numpy(st.queries.view(np.int16).copy()).view(torch.bfloat16).float().mean(0).to(torch.bfloat16)
    st.cache_vecs[first:first + 150] = mean.view(torch.int16).numpy().view(np.uint16)[None, :]
    ref = fo.lookup(st.queries[:8], st.cache_vecs, st.cache_labels, k=k, tau=0.0)
    np.testing.assert_array_equal(ref.ni, np.tile(np.arange(first, first + k), (8, 1)))   # the premise, by the oracle
    cache = make_cache(st, k=k, num_classes=1, tau=0.0, max_batch=b, path=fb.FI_PATH_GEMM)
    got = run_lookup(cache, st.queries)
    np.testing.assert_array_equal(got[4], np.tile(np.arange(first, first + k, dtype=np.int32), (b, 1)))
    assert (got[3] == got[3][:, :1]).all()
    np.testing.assert_allclose(got[3][:8], ref.nd, rtol=2e-3)
    cache.close()


def test_tensor_core_and_streaming_paths_agree_on_random_deep_shapes():
    """Consistency, not parity (no oracle here): on 16 seeded random shapes of deep rows (4,096-16,384 values, 129-900
    requests behind a gather list, a device-resident count, sometimes an SM limit) the tensor-core path, whose work split
    changes form with every one of these numbers, returns the neighbours and distances of the streaming path, which
    computes every distance directly.  A differing neighbour set is accepted only for a tie at the k-th place."""
    rng = np.random.default_rng(7)
    forms = set()
    fixed = [(8192, 800, 11700, 13, 800, 0), (16384, 600, 20, 5, 600, 0)]   # wave + tail; ranges over a handful of rows
    for case in range(16):
        d = int(rng.choice([4096, 4160, 8192, 16384]))
        b = int(rng.integers(129, 900))
        n = int(rng.choice([rng.integers(1, 40), rng.integers(40, 600), rng.integers(600, 12000)]))
        k = int(rng.choice([1, 5, 13, 29]))
        count = int(rng.integers(1, b + 1)) if rng.random() < 0.6 else b
        sms = int(rng.choice([0, 0, 100, 37, 8]))
        if case < len(fixed):
            d, b, n, k, count, sms = fixed[case]
        w = dg.single_layer(name="f", n_cache=n, n_query=b, dim=d, num_classes=7, dtype="bf16", sigma=0.6, k=k,
                            seed=int(rng.integers(1 << 30)))
        st = w.stages[0]
        forms.add(fb.gemm_plan_describe(count, n, sms or 148, k, d, b)[0]["mode"])
        perm = torch.from_numpy(rng.permutation(b).astype(np.int32)).to("cuda:0")
        cnt = torch.tensor([count], dtype=torch.int32, device="cuda:0")
        res = []
        for path in (fb.FI_PATH_STREAM, fb.FI_PATH_GEMM):
            c = make_cache(st, k=k, num_classes=7, tau=0.0, max_batch=b + 100, path=path)
            if sms:
                c.set_sm_limit(sms)
            out = c.lookup_batch(to_device(st.queries), row_idx=perm, batch_max=b, batch_count=cnt)
            torch.cuda.synchronize()
            c.poll_status()
            res.append((out.topk_dist.cpu().numpy()[:count], out.topk_idx.cpu().numpy()[:count]))
            c.close()
        (d0, i0), (d1, i1) = res
        ke = min(k, n)
        np.testing.assert_allclose(d1[:, :ke], d0[:, :ke], rtol=2e-3)
        for r in range(count):
            if set(i0[r, :ke]) != set(i1[r, :ke]):
                assert abs(d0[r, ke - 1] - d1[r, ke - 1]) <= 1e-4 * d0[r, ke - 1], (d, b, n, k, count, sms, r)
    assert forms == {0, 1, 3}


def test_gemm_and_stream_paths_agree_and_copies_hit():
    w = dg.single_layer(name="t", n_cache=3000, n_query=40, dim=512, num_classes=6, dtype="bf16", sigma=0.5, k=5,
                        seed=6, n_copies=8)
    st = w.stages[0]
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=5, tau=1e30)
    outs = []
    for path in (fb.FI_PATH_STREAM, fb.FI_PATH_GEMM):
        cache = make_cache(st, k=5, num_classes=6, tau=1e30, max_batch=48, path=path)
        got = run_lookup(cache, st.queries)
        compare_lookup(*got, ref, storage="bf16", tau=1e30, rule=0, cache_labels=st.cache_labels)
        outs.append(got)
        cache.close()
    copies = w.meta["copy_of"] >= 0
    for got in outs:   # observation O1: an identical activation freezes, whatever the threshold
        assert (got[3][copies, 0] == 0).all() and np.isinf(got[1][copies]).all() and (got[2][copies] == 1).all()
        assert (got[2][~copies] == 0).all()
    np.testing.assert_array_equal(outs[0][0], outs[1][0])
    np.testing.assert_array_equal(outs[0][4], outs[1][4])


def test_kmeans_entries_weights_and_l2_metric():
    # Sec. 4: entries <centre, majority label, fraction>; k = 1 gives confidence f / distance
    w = dg.single_layer(name="t", n_cache=200, n_query=64, dim=1024, num_classes=10, dtype="bf16", sigma=0.5, k=1, seed=7)
    frac = np.random.default_rng(0).uniform(0.4, 1.0, 200).astype(np.float32)
    for path in (fb.FI_PATH_STREAM, fb.FI_PATH_GEMM):
        for metric in (0, 1):
            check_case(w.stages[0], k=1, num_classes=10, rule=fo.RULE_CONF_GT, path=path, metric=metric, weights=frac)
    check_case(w.stages[0], k=4, num_classes=10, rule=fo.RULE_DIST_LE, path=fb.FI_PATH_GEMM, metric=1, weights=frac)


@pytest.mark.parametrize("n,d,b,k,rule,metric,weighted", [
    (3000, 64, 8200, 5, fo.RULE_CONF_GT, 0, False),     # the paper's vote, several labels among the neighbours
    (200, 1024, 9000, 1, fo.RULE_CONF_GT, 1, True),     # k-means cache: k = 1, weights, L2 metric
    (1500, 200, 8500, 13, fo.RULE_DIST_LE, 0, True),    # list length 16, distance rule
    (700, 136, 8192, 29, fo.RULE_CONF_GT, 0, False),    # too many candidate entries for a warp: CTA per query
    (200, 1024, 8200, 29, fo.RULE_CONF_GT, 0, False),   # 32 candidates per query: every lane of the warp holds one
    (200, 1024, 19000, 1, fo.RULE_CONF_GT, 1, True),    # 75 query tiles on one cache-row tile: dealt round-robin to the CTAs
    (250, 64, 9500, 5, fo.RULE_CONF_GT, 0, False),      # the same with 128-query tiles (two lists per query)
])
def test_large_batches_of_short_rows(n, d, b, k, rule, metric, weighted):
    """Batches of 8,192 and more against rows of at most 8 KiB are finished one query per warp."""
    w = dg.single_layer(name="t", n_cache=n, n_query=b, dim=d, num_classes=7, dtype="bf16", sigma=0.6, k=k, seed=21)
    weights = np.random.default_rng(3).uniform(0.3, 1.0, n).astype(np.float32) if weighted else None
    check_case(w.stages[0], k=k, num_classes=7, rule=rule, path=fb.FI_PATH_GEMM, metric=metric, weights=weights)


def test_large_batch_fp32_streaming_lists():
    """The same finish on the streaming kernel's candidate lists (fp32 cache, exact distances, no re-ranking)."""
    w = dg.single_layer(name="t", n_cache=300, n_query=8300, dim=32, num_classes=5, dtype="f32", sigma=0.5, k=3, seed=22)
    check_case(w.stages[0], k=3, num_classes=5, rule=fo.RULE_CONF_GT, path=fb.FI_PATH_STREAM)


# ------------------------------------------------------------------ degenerate cases

def test_empty_cache_k_above_size_and_zero_batch():
    w = dg.single_layer(name="t", n_cache=3, n_query=6, dim=64, num_classes=4, dtype="bf16", sigma=0.5, k=5, seed=8)
    st = w.stages[0]
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=5, tau=0.0)
    for path in (fb.FI_PATH_STREAM, fb.FI_PATH_GEMM):
        cache = make_cache(st, k=5, num_classes=4, tau=0.0, max_batch=8, path=path, capacity=10)
        got = run_lookup(cache, st.queries)
        compare_lookup(*got, ref, storage="bf16", tau=0.0, rule=0, cache_labels=st.cache_labels)
        assert (got[4][:, 3:] == -1).all()
        cache.close()
    empty = fb.FreezeCache(dim=64, capacity=10, num_classes=4, k=5, dtype=fb.FI_BF16, max_batch=8)
    got = run_lookup(empty, st.queries)
    assert (got[0] == -1).all() and (got[1] == 0).all() and (got[2] == 0).all() and (got[4] == -1).all()
    # batch 0: nothing is launched, nothing is written
    q = to_device(st.queries, empty.device)
    out = fb.LookupOut(1, 5, empty.device)
    out.label.fill_(77)
    empty.lookup_batch(q[:0], batch_max=0, out=out)
    torch.cuda.synchronize()
    assert int(out.label[0]) == 77
    empty.close()


def test_gather_list_and_device_resident_count():
    w = dg.single_layer(name="t", n_cache=2000, n_query=300, dim=256, num_classes=5, dtype="bf16", sigma=0.5, k=5, seed=9)
    st = w.stages[0]
    rows = np.sort(np.random.default_rng(1).choice(300, 150, replace=False)).astype(np.int32)
    for path, count in ((fb.FI_PATH_GEMM, 131), (fb.FI_PATH_STREAM, 3), (fb.FI_PATH_GEMM, 0)):
        cache = make_cache(st, k=5, num_classes=5, tau=0.05, max_batch=150, path=path)
        ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=5, tau=f32(0.05), row_idx=rows[:count])
        out = fb.LookupOut(150, 5, cache.device)
        out.label.fill_(-7)
        cnt = torch.tensor([count], dtype=torch.int32, device=cache.device)
        cache.lookup_batch(to_device(st.queries, cache.device), row_idx=torch.from_numpy(rows).to(cache.device),
                           batch_max=150, batch_count=cnt, out=out)
        torch.cuda.synchronize()
        cache.poll_status()
        lab = out.label.cpu().numpy()
        assert (lab[count:] == -7).all()      # slots past the actual batch stay untouched
        if count:
            compare_lookup(lab[:count], out.conf.cpu().numpy()[:count], out.hit.cpu().numpy()[:count],
                           out.topk_dist.cpu().numpy()[:count], out.topk_idx.cpu().numpy()[:count], ref, storage="bf16",
                           tau=f32(0.05), rule=0, cache_labels=st.cache_labels)
        cache.close()


def test_strided_queries_and_incremental_insert():
    w = dg.single_layer(name="t", n_cache=900, n_query=20, dim=128, num_classes=5, dtype="bf16", sigma=0.5, k=3, seed=10)
    st = w.stages[0]
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=3, tau=0.0)
    for path in (fb.FI_PATH_STREAM, fb.FI_PATH_GEMM):
        cache = fb.FreezeCache(dim=128, capacity=1000, num_classes=5, k=3, dtype=fb.FI_BF16, max_batch=32, path=path)
        xs, ls = to_device(st.cache_vecs), torch.from_numpy(st.cache_labels).cuda()
        for lo, hi in ((0, 1), (1, 450), (450, 900)):     # Sec. 5: entries can be appended later
            cache.insert(xs[lo:hi].contiguous(), ls[lo:hi].contiguous())
        assert cache.size() == 900
        wide = torch.zeros(20, 256, dtype=torch.bfloat16, device="cuda")
        wide[:, :128] = to_device(st.queries)
        out = cache.lookup_batch(wide[:, :128])              # leading dimension 256
        torch.cuda.synchronize()
        compare_lookup(out.label.cpu().numpy(), out.conf.cpu().numpy(), out.hit.cpu().numpy(),
                       out.topk_dist.cpu().numpy(), out.topk_idx.cpu().numpy(), ref, storage="bf16", tau=0.0, rule=0,
                       cache_labels=st.cache_labels)
        cache.close()


def test_error_statuses():
    with pytest.raises(fb.FiError) as e:
        fb.FreezeCache(dim=12, capacity=10, num_classes=4, k=5, dtype=fb.FI_BF16)      # dim not a multiple of 8
    assert e.value.status == 1
    with pytest.raises(fb.FiError) as e:
        fb.FreezeCache(dim=16, capacity=10, num_classes=4, k=33, dtype=fb.FI_BF16)     # k above 32
    assert e.value.status == 1
    with pytest.raises(fb.FiError) as e:
        fb.FreezeCache(dim=16, capacity=10, num_classes=4, k=3, dtype=fb.FI_F32, path=fb.FI_PATH_GEMM)
    assert e.value.status == 5
    c = fb.FreezeCache(dim=16, capacity=4, num_classes=4, k=1, dtype=fb.FI_BF16, max_batch=4)
    x = torch.zeros(5, 16, dtype=torch.bfloat16, device="cuda")
    lab = torch.zeros(5, dtype=torch.int32, device="cuda")
    with pytest.raises(fb.FiError) as e:
        c.insert(x, lab)                                                                  # beyond capacity
    assert e.value.status == 2 and c.size() == 0
    with pytest.raises(fb.FiError) as e:
        c.lookup_batch(x)                                                                 # batch above max_batch
    assert e.value.status == 1
    c.close()


# ------------------------------------------------------------------ cascades

def oracle_taus(w):
    taus = []
    for s, p in zip(w.stages, w.meta["percentiles"]):
        c = fo.lookup(s.calib, s.cache_vecs, s.cache_labels, k=w.k, tau=0.0).conf
        taus.append(f32(np.percentile(c, p)))
    return taus


def run_cascade_device(w, taus, path):
    b0 = w.stages[0].queries.shape[0]
    caches = [make_cache(s, k=w.k, num_classes=w.num_classes, tau=t, max_batch=b0, path=path)
              for s, t in zip(w.stages, taus)]
    acts = [to_device(s.queries) for s in w.stages]
    state = fb.CascadeState(b0, "cuda:0")
    fb.cascade_init(state, len(caches))
    survivors = []
    for l, (c, a) in enumerate(zip(caches, acts)):
        fb.cascade_step(c, a, state, l)
        ids, cnt = state.survivors(l)
        torch.cuda.synchronize()
        survivors.append(ids[: int(cnt.item())].cpu().numpy().copy())
    for c in caches:
        c.poll_status()
    res = (state.final_label.cpu().numpy()[:b0], state.exit_stage.cpu().numpy()[:b0],
           state.final_conf.cpu().numpy()[:b0], survivors)
    return caches, res


def check_cascade(w, path):
    taus = oracle_taus(w)
    ref = fo.cascade([s.queries for s in w.stages], [s.cache_vecs for s in w.stages],
                     [s.cache_labels for s in w.stages], taus, k=w.k)
    caches, (label, stage, conf, survivors) = run_cascade_device(w, taus, path)
    stats = compare_cascade(ref, taus, label, stage, conf, survivors, stage_labels=[s.cache_labels for s in w.stages])
    print(f"{w.name}: {stats}")
    assert stats.mismatches == 0
    assert ref.active[-1].shape[0] > 0 and (ref.exit_stage == 0).sum() > 0
    # the host-buffer entry point gives the same answers
    from helpers import to_host_tensor
    b0 = label.shape[0]
    hl = torch.empty(b0, dtype=torch.int32).pin_memory()
    hs = torch.empty(b0, dtype=torch.int32).pin_memory()
    hc = torch.empty(b0, dtype=torch.float32).pin_memory()
    arr = torch.zeros(len(caches) + 1, dtype=torch.int32).pin_memory()
    fb.cascade_run_host(caches, [to_host_tensor(s.queries, pin=True) for s in w.stages], hl, hs, hc, arr)
    np.testing.assert_array_equal(hl.numpy(), label)
    np.testing.assert_array_equal(hs.numpy(), stage)
    np.testing.assert_array_equal(hc.numpy(), conf)
    np.testing.assert_array_equal(arr.numpy(), [b0] + [s.shape[0] for s in survivors])
    for c in caches:
        c.close()


@pytest.mark.parametrize("path", [fb.FI_PATH_GEMM, fb.FI_PATH_STREAM])
def test_cascade_resnet18_shape_shrunk(path):
    check_cascade(dg.config2(seed=0, shrink=16), path)


def test_cascade_imagenet_shape_shrunk():
    check_cascade(dg.config4(seed=0, shrink=8), fb.FI_PATH_GEMM)


def test_cascade_of_deep_rows_whose_batch_shrinks_below_half_a_tile():
    # 600 requests (three 256-row tiles, the last at most half full at some stage) down to fewer than 128 (one half
    # tile) against rows of 4,096 values: every stage runs the spans form of the distance GEMM
    w = dg.cascade(name="t", dims=[4096, 4096, 4096, 4096], scales=[0.2, 0.4, 0.8, 1.6], kind="halfnormal", n_cache=1500,
                   n_query=600, n_calib=128, num_classes=10, dtype="bf16", k=5, seed=5)
    w.meta.update(rule="conf_gt", percentiles=[45.0, 40.0, 40.0, 40.0])
    check_cascade(w, fb.FI_PATH_GEMM)


def test_cascade_threshold_limits():
    w = dg.config2(seed=0, shrink=32)
    _, (label, stage, _, surv) = run_cascade_device(w, [float("inf")] * 4, fb.FI_PATH_GEMM)
    assert (stage == 4).all() and (label == -1).all() and all(s.shape[0] == 32 for s in surv)
    _, (label, stage, _, surv) = run_cascade_device(w, [0.0] * 4, fb.FI_PATH_GEMM)
    assert (stage == 0).all() and all(s.shape[0] == 0 for s in surv)


def test_host_lookup_matches_device_lookup():
    from helpers import to_host_tensor
    w = dg.single_layer(name="t", n_cache=1200, n_query=70, dim=256, num_classes=5, dtype="bf16", sigma=0.5, k=5, seed=12)
    st = w.stages[0]
    cache = make_cache(st, k=5, num_classes=5, tau=0.02, max_batch=70)
    dev = run_lookup(cache, st.queries)
    out = fb.LookupOut(70, 5, "cpu")
    cache.lookup_batch_host(to_host_tensor(st.queries, pin=True), out)
    for a, b in zip(dev, (out.label, out.conf, out.hit, out.topk_dist, out.topk_idx)):
        np.testing.assert_array_equal(a, b.numpy())
    cache.close()


# ------------------------------------------------------------------ ComputeThresholds on the device

@pytest.mark.parametrize("path,max_batch", [(fb.FI_PATH_GEMM, 64), (fb.FI_PATH_STREAM, 200)])
def test_compute_threshold_matches_oracle(path, max_batch):
    w = dg.single_layer(name="t", n_cache=1500, n_query=200, dim=256, num_classes=8, dtype="bf16", sigma=0.9, k=3,
                        seed=15)
    st = w.stages[0]
    # stand-in for the label the model predicts per item: the item's class, for 15 % of the items another one, so
    # that some look-ups disagree with "the model" as they do on real validation data
    flip = np.random.default_rng(16).random(200) < 0.15
    model = np.where(flip, (w.query_classes + 1) % 8, w.query_classes).astype(np.int32)
    want_tau, want_wrong = fo.compute_threshold(st.queries, st.cache_vecs, st.cache_labels, model, k=3)
    cache = make_cache(st, k=3, num_classes=8, tau=123.0, max_batch=max_batch, path=path)    # 200 items: several batches
    tau, wrong = cache.compute_threshold(to_device(st.queries), torch.from_numpy(model).cuda())
    assert wrong == want_wrong and 0 < wrong < 200
    assert tau == pytest.approx(want_tau, rel=1e-5)
    # the cache now freezes no validation item wrongly
    first = min(200, max_batch)
    out = cache.lookup_batch(to_device(st.queries[:first]))
    torch.cuda.synchronize()
    hit = out.hit.cpu().numpy() == 1
    assert hit.any() and (out.label.cpu().numpy()[hit] == model[:first][hit]).all()
    cache.close()


# ------------------------------------------------------------------ failure path: a wait that runs out

def test_bounded_wait_reports_timeout_and_context_survives():
    w = dg.single_layer(name="t", n_cache=500, n_query=40, dim=128, num_classes=5, dtype="bf16", sigma=0.5, k=3, seed=17)
    st = w.stages[0]
    cache = make_cache(st, k=3, num_classes=5, tau=0.0, max_batch=40, path=fb.FI_PATH_GEMM)
    before = run_lookup(cache, st.queries)
    cache.selftest_wait(2_000_000)                       # about a millisecond on a barrier nothing completes
    with pytest.raises(fb.FiError) as e:
        cache.poll_status()
    assert e.value.status == 6 and "bounded wait" in str(e.value)
    cache.poll_status()                                   # the word was cleared by the poll that reported it
    after = run_lookup(cache, st.queries)                 # same device, same context, same answers
    for a, b in zip(before, after):
        np.testing.assert_array_equal(a, b)
    cache.close()


def test_host_entry_points_report_a_timed_out_wait():
    """A call that synchronises anyway returns FI_ERR_TIMEOUT itself when a kernel of one of its caches gave up on a
    bounded wait, instead of handing back results nobody should trust; the word is cleared and the next call is clean."""
    from helpers import to_host_tensor
    w = dg.config2(seed=0, shrink=32)
    b0 = w.stages[0].queries.shape[0]
    caches = [make_cache(s, k=w.k, num_classes=w.num_classes, tau=1e-3, max_batch=b0) for s in w.stages]
    acts = [to_host_tensor(s.queries, pin=True) for s in w.stages]
    hl = torch.empty(b0, dtype=torch.int32).pin_memory()
    hs = torch.empty(b0, dtype=torch.int32).pin_memory()
    hc = torch.empty(b0, dtype=torch.float32).pin_memory()
    fb.cascade_run_host(caches, acts, hl, hs, hc)
    want = (hl.clone(), hs.clone(), hc.clone())
    caches[2].selftest_wait(2_000_000)                    # a wait that nothing completes, about a millisecond long
    with pytest.raises(fb.FiError) as e:
        fb.cascade_run_host(caches, acts, hl, hs, hc)
    assert e.value.status == 6 and "bounded wait" in str(e.value)
    fb.cascade_run_host(caches, acts, hl, hs, hc)         # cleared by the call that reported it
    for a, b in zip(want, (hl, hs, hc)):
        assert torch.equal(a, b)
    out = fb.LookupOut(b0, w.k, "cpu")
    caches[0].selftest_wait(2_000_000)
    with pytest.raises(fb.FiError) as e:
        caches[0].lookup_batch_host(acts[0], out)
    assert e.value.status == 6
    caches[0].lookup_batch_host(acts[0], out)
    caches[1].selftest_wait(2_000_000)
    with pytest.raises(fb.FiError) as e:
        caches[1].compute_threshold(to_device(w.stages[1].queries), torch.zeros(b0, dtype=torch.int32, device="cuda"))
    assert e.value.status == 6
    for c in caches:
        c.poll_status()
        c.close()


def test_partly_filled_cache_never_outgrows_the_scratch_sized_at_create():
    """The tile plan is not monotone in the number of entries: a cache holding a fraction of its capacity can cut more
    ranges, hence more candidate lists per request, than the full one.  The scratch allocated at create covers every
    fill level, so look-ups at every level run (and match the oracle) without allocating."""
    w = dg.single_layer(name="t", n_cache=6000, n_query=700, dim=128, num_classes=5, dtype="bf16", sigma=0.6, k=5, seed=31)
    st = w.stages[0]
    cache = fb.FreezeCache(dim=128, capacity=6000, num_classes=5, k=5, dtype=fb.FI_BF16, max_batch=700, path=fb.FI_PATH_GEMM)
    xs, ls, q = to_device(st.cache_vecs), torch.from_numpy(st.cache_labels).cuda(), to_device(st.queries)
    free_before = None
    filled = 0
    for upto in (40, 300, 1200, 2400, 6000):
        cache.insert(xs[filled:upto].contiguous(), ls[filled:upto].contiguous())
        filled = upto
        out = cache.lookup_batch(q)
        torch.cuda.synchronize()
        if free_before is None:
            free_before = torch.cuda.mem_get_info()[0]
        ref = fo.lookup(st.queries, st.cache_vecs[:upto], st.cache_labels[:upto], k=5, tau=0.0)
        compare_lookup(out.label.cpu().numpy(), out.conf.cpu().numpy(), out.hit.cpu().numpy(), out.topk_dist.cpu().numpy(),
                       out.topk_idx.cpu().numpy(), ref, storage="bf16", tau=0.0, rule=0, cache_labels=st.cache_labels[:upto])
    cache.poll_status()
    cache.close()


def test_caches_created_from_two_threads():
    """Kernel set-up is per device and locked: two threads creating caches and looking up at the same time both work."""
    import threading
    w = dg.single_layer(name="t", n_cache=900, n_query=150, dim=256, num_classes=5, dtype="bf16", sigma=0.5, k=5, seed=33)
    st = w.stages[0]
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=5, tau=0.0)
    results, errors = {}, []

    def work(tid):
        try:
            with torch.cuda.stream(torch.cuda.Stream()):
                for rep in range(3):
                    c = make_cache(st, k=5, num_classes=5, tau=0.0, max_batch=150, path=fb.FI_PATH_GEMM)
                    out = c.lookup_batch(to_device(st.queries))
                    torch.cuda.current_stream().synchronize()
                    results[(tid, rep)] = [t.cpu().numpy() for t in (out.label, out.conf, out.hit, out.topk_dist, out.topk_idx)]
                    c.poll_status()
                    c.close()
        except Exception as exc:                          # pragma: no cover
            errors.append(exc)

    threads = [threading.Thread(target=work, args=(t,)) for t in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert len(results) == 6
    for got in results.values():
        compare_lookup(*got, ref, storage="bf16", tau=0.0, rule=0, cache_labels=st.cache_labels)


# ------------------------------------------------------------------ inserts into a cache that is being looked up

@pytest.mark.parametrize("path", [fb.FI_PATH_GEMM, fb.FI_PATH_STREAM])
def test_inserts_on_one_stream_while_lookups_run_on_another(path):
    """Sec. 5, incremental cache update.  Entries are appended on one stream while look-ups run on another; every look-up
    covers a prefix of the entries (reported by lookup_view) and must equal the oracle's answer on exactly that prefix."""
    n, chunk, d, b, k = 24000, 3000, 2048, 48, 5
    w = dg.single_layer(name="t", n_cache=n, n_query=b, dim=d, num_classes=6, dtype="bf16", sigma=0.6, k=k, seed=51)
    st = w.stages[0]
    cache = fb.FreezeCache(dim=d, capacity=n, num_classes=6, k=k, dtype=fb.FI_BF16, max_batch=b, path=path)
    xs, ls, q = to_device(st.cache_vecs), torch.from_numpy(st.cache_labels).cuda(), to_device(st.queries)
    s_ins, s_look = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    seen = []
    for lo in range(0, n, chunk):
        with torch.cuda.stream(s_ins):
            cache.insert(xs[lo:lo + chunk], ls[lo:lo + chunk])
        assert cache.size() == lo + chunk                      # enqueued entries count at once
        with torch.cuda.stream(s_look):
            out = cache.lookup_batch(q)
            seen.append((cache.lookup_view(), out))
    torch.cuda.synchronize()
    out = cache.lookup_batch(q)                                # everything has landed: the whole cache
    seen.append((cache.lookup_view(), out))
    torch.cuda.synchronize()
    cache.poll_status()
    views = [v for v, _ in seen]
    print(f"path {path}: look-ups covered {views} entries while {n // chunk} inserts of {chunk} were enqueued")
    assert views == sorted(views) and views[-1] == n and all(v % chunk == 0 for v in views)
    assert all(v <= (i + 1) * chunk for i, v in enumerate(views[:-1]))
    refs = {}
    for view, out in seen:
        got = [t.cpu().numpy() for t in (out.label, out.conf, out.hit, out.topk_dist, out.topk_idx)]
        if view == 0:
            assert (got[0] == -1).all() and (got[2] == 0).all() and (got[4] == -1).all()
            continue
        if view not in refs:
            refs[view] = fo.lookup(st.queries, st.cache_vecs[:view], st.cache_labels[:view], k=k, tau=0.0)
        compare_lookup(*got, refs[view], storage="bf16", tau=0.0, rule=0, cache_labels=st.cache_labels[:view])
    cache.close()


def test_lookup_on_a_limited_number_of_sms_gives_the_same_answers():
    w = dg.single_layer(name="t", n_cache=9000, n_query=600, dim=1024, num_classes=6, dtype="bf16", sigma=0.6, k=5, seed=52)
    st = w.stages[0]
    cache = make_cache(st, k=5, num_classes=6, tau=0.0, max_batch=600)
    full = run_lookup(cache, st.queries)
    for sms in (40, 7):
        cache.set_sm_limit(sms)
        part = run_lookup(cache, st.queries)
        for a, c in zip(full, part):
            np.testing.assert_array_equal(a, c)
    cache.set_sm_limit(0)
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=5, tau=0.0)
    compare_lookup(*full, ref, storage="bf16", tau=0.0, rule=0, cache_labels=st.cache_labels)
    cache.close()


# ------------------------------------------------------------------ certificate of the tensor-core path, exact repair

def _near_duplicate_case(n, d, b, seed):
    """Cache rows and requests that are all small perturbations of one vector of large entries: ||q||^2 is about 1e4
    times the distances, so the rounding of the tensor-core scores is of the order of the gaps between neighbours."""
    rng = np.random.default_rng(seed)
    base = 64.0 + 0.5 * rng.integers(0, 8, size=d)                    # exactly representable in bf16 (step 0.5 here)
    x = (base[None, :] + 0.5 * rng.integers(-2, 3, size=(n, d))).astype(np.float32)
    q = (base[None, :] + 0.5 * rng.integers(-2, 3, size=(b, d))).astype(np.float32)
    labels = rng.integers(0, 4, size=n).astype(np.int32)
    from paper_2002_02645_b200.datagen import StageData, f32_to_bf16_bits
    xb, qb = f32_to_bf16_bits(x), f32_to_bf16_bits(q)
    assert (dg.bf16_bits_to_f32(xb) == x).all() and (dg.bf16_bits_to_f32(qb) == q).all()
    return StageData(d, "bf16", xb, labels, qb)


def test_certificate_marks_undecidable_requests_and_repair_makes_them_exact():
    st = _near_duplicate_case(n=12000, d=1024, b=160, seed=41)
    k = 5
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=k, tau=0.0)
    cache = make_cache(st, k=k, num_classes=4, tau=0.0, max_batch=160, path=fb.FI_PATH_GEMM)
    cache.read_certificate()                                         # clears whatever the set-up left
    got = run_lookup(cache, st.queries)
    flags = cache.slot_certificates(160).numpy().astype(bool)
    uncertified, unrepaired, err = cache.read_certificate()
    eps = (1024 / 16 + 4) * 2.0 ** -23
    print(f"near-duplicate rows: {uncertified} of 160 requests without a certificate, largest score error {err:.3g} "
          f"(bound used {eps:.3g})")
    assert uncertified == int((~flags).sum()) == unrepaired and 0 < uncertified <= 160
    assert 0 < err <= eps                                            # the error model holds on the candidates seen
    # certified requests are proven exact: they must equal the oracle (the k-th gap exemption apart)
    sub = np.nonzero(flags)[0]
    from oracle.fi_oracle import LookupResult
    pick = lambda r, i: LookupResult(r.label[i], r.conf[i], r.hit[i], r.nd[i], r.ni[i], r.next_d[i])
    compare_lookup(*[g[sub] for g in got], pick(ref, sub), storage="bf16", tau=0.0, rule=0, cache_labels=st.cache_labels)
    # with the repair pass every request is either certified or looked up again with exact distances
    cache.set_repair(True)
    fixed = run_lookup(cache, st.queries)
    flags2 = cache.slot_certificates(160).numpy().astype(bool)
    unc2, unrep2, _ = cache.read_certificate()
    assert unc2 == uncertified and unrep2 == max(0, uncertified - 64)
    assert int((~flags2).sum()) == unrep2
    sub2 = np.nonzero(flags2)[0]
    stats = compare_lookup(*[g[sub2] for g in fixed], pick(ref, sub2), storage="bf16", tau=0.0, rule=0,
                           cache_labels=st.cache_labels)
    print(stats)
    again = run_lookup(cache, st.queries)
    for a, b2 in zip(fixed, again):
        np.testing.assert_array_equal(a, b2)
    cache.close()


def test_certificate_on_ordinary_data_and_streaming_path():
    w = dg.single_layer(name="t", n_cache=5000, n_query=300, dim=512, num_classes=6, dtype="bf16", sigma=0.6, k=5, seed=43)
    st = w.stages[0]
    for path in (fb.FI_PATH_GEMM, fb.FI_PATH_STREAM):
        cache = make_cache(st, k=5, num_classes=6, tau=0.0, max_batch=300, path=path)
        cache.read_certificate()
        run_lookup(cache, st.queries)
        unc, unrep, err = cache.read_certificate()
        flags = cache.slot_certificates(300).numpy()
        print(f"path {path}: uncertified {unc}, largest score error {err:.3g}")
        assert unc == int((flags == 0).sum())
        if path == fb.FI_PATH_STREAM:
            assert unc == 0 and err == 0.0                          # exact distances throughout: nothing to certify
        else:
            assert unc < 150 and 0 < err <= (512 / 16 + 4) * 2.0 ** -23
        cache.close()


# ------------------------------------------------------------------ cache rows split over several caches (shards)

@pytest.mark.parametrize("path", [fb.FI_PATH_GEMM, fb.FI_PATH_STREAM])
def test_row_sharded_lookup_matches_unsharded_oracle(path):
    """Three shards stand in for three GPUs: each answers from its rows, the tuples are pooled as an all-gather would
    deliver them, and every "rank" merges them with fi_merge_shard_lookups."""
    from paper_2002_02645_b200.datagen import StageData
    w = dg.single_layer(name="t", n_cache=3000, n_query=96, dim=512, num_classes=6, dtype="bf16", sigma=0.5, k=5, seed=25)
    st = w.stages[0]
    ref0 = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=5, tau=0.0)
    tau = f32(np.median(ref0.conf))
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=5, tau=tau)
    cuts = [0, 1000, 1003, 3000]
    q = to_device(st.queries)
    gathered = [[], [], [], []]
    for a, b in zip(cuts, cuts[1:]):
        shard = StageData(st.dim, "bf16", st.cache_vecs[a:b], st.cache_labels[a:b], st.queries)
        c = make_cache(shard, k=5, num_classes=6, tau=tau, max_batch=96, path=path)
        out = c.lookup_batch(q)
        gi, lab, wgt = c.neighbor_tuples(out.topk_idx, a)
        torch.cuda.synchronize()
        for lst, t in zip(gathered, (out.topk_dist, gi, lab, wgt)):
            lst.append(t.clone())
        c.close()
    merged = fb.merge_shard_lookups(*[torch.stack(g) for g in gathered], threshold=tau)
    torch.cuda.synchronize()
    compare_lookup(merged.label.cpu().numpy(), merged.conf.cpu().numpy(), merged.hit.cpu().numpy(),
                   merged.topk_dist.cpu().numpy(), merged.topk_idx.cpu().numpy(), ref, storage="bf16", tau=tau, rule=0,
                   cache_labels=st.cache_labels)
    assert 0 < ref.hit.sum() < 96
