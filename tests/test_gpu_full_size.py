"""The five workloads at their full sizes, in the launch configuration bench.py times.

The GPU serves every request; the fp64 oracle is run on a sample of the requests (a request's way through the
cascade does not depend on the other requests of the batch, so the oracle's answers for a subset are the answers
it would give inside the full batch).  What cannot be sampled is checked through properties that hold at any size:
survivor lists ascending, counts consistent with the exit stages, frozen + surviving = batch.
"""
import numpy as np
import pytest
import torch

from oracle import fi_oracle as fo
from paper_2002_02645_b200 import binding as fb
from paper_2002_02645_b200 import datagen as dg
from helpers import compare_cascade, compare_lookup, f32, make_cache, to_device

pytestmark = pytest.mark.gpu


def calibrated_taus(w, caches):
    """Thresholds as bench.py sets them: percentile of the library's own confidences on the calibration batch."""
    taus = []
    for c, s, p in zip(caches, w.stages, w.meta["percentiles"]):
        c.set_threshold(0.0)
        conf = c.lookup_batch(to_device(s.calib), with_topk=False).conf.cpu().numpy().astype(np.float64)
        tau = f32(np.percentile(conf[np.isfinite(conf)], p))
        c.set_threshold(tau)
        taus.append(tau)
    return taus


def run_full_cascade(w, sample_ids):
    b0 = w.stages[0].queries.shape[0]
    caches = [make_cache(s, k=w.k, num_classes=w.num_classes, tau=0.0,
                         max_batch=max(b0, s.calib.shape[0])) for s in w.stages]
    taus = calibrated_taus(w, caches)
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
    label = state.final_label.cpu().numpy()[:b0]
    stage = state.exit_stage.cpu().numpy()[:b0]
    conf = state.final_conf.cpu().numpy()[:b0]
    n_stage = len(caches)
    # ---- properties at full size
    alive = np.arange(b0)
    for l in range(n_stage):
        s = survivors[l]
        assert (np.diff(s) > 0).all()
        np.testing.assert_array_equal(s, alive[stage[alive] > l])       # survivors = requests not frozen up to l
        alive = s
    assert ((stage == n_stage) == (label == -1)).all()
    assert sum((stage == l).sum() for l in range(n_stage + 1)) == b0
    # ---- oracle on the sample
    ref = fo.cascade([s.queries[sample_ids] for s in w.stages], [s.cache_vecs for s in w.stages],
                     [s.cache_labels for s in w.stages], taus, k=w.k)
    stats = compare_cascade(ref, taus, label, stage, conf, survivors, sample_ids=sample_ids,
                            stage_labels=[s.cache_labels for s in w.stages])
    # distances concentrate in these dimensions, so many requests meet a k-th/(k+1)-th gap below 1e-4 somewhere on
    # their way; from that stage on they are exempt from the bit-exact rule and counted (in practice still equal)
    print(f"{w.name}: full-batch arrivals {[b0] + [s.shape[0] for s in survivors]}, oracle sample: {stats}")
    assert stats.mismatches == 0
    assert stats.exempt - stats.exempt_equal_anyway <= max(1, len(sample_ids) // 20)   # exempt requests rarely differ at all
    assert all(s.shape[0] > 0 for s in survivors) and (stage == 0).sum() > 0
    for c in caches:
        c.close()


def test_config2_full_cascade():
    w = dg.config2(seed=0)
    run_full_cascade(w, np.arange(0, 1024, 16))            # 64 requests through the oracle


def test_config4_full_cascade():
    w = dg.config4(seed=0)
    run_full_cascade(w, np.arange(0, 4096, 32))            # 128 requests through the oracle


def test_config3_full_lookup():
    w = dg.config3(seed=0)
    st = w.stages[0]
    cache = make_cache(st, k=10, num_classes=10, tau=0.0, max_batch=8192)
    tau = calibrated_taus(w, [cache])[0]
    out = cache.lookup_batch(to_device(st.queries))
    torch.cuda.synchronize()
    cache.poll_status()
    got = [t.cpu().numpy() for t in (out.label, out.conf, out.hit, out.topk_dist, out.topk_idx)]
    sample = np.arange(0, 8192, 64)                         # 128 requests against all 200,000 entries
    ref = fo.lookup(st.queries[sample], st.cache_vecs, st.cache_labels, k=10, tau=tau)
    stats = compare_lookup(*[g[sample] for g in got], ref, storage="bf16", tau=tau, rule=0,
                           cache_labels=st.cache_labels)
    print(stats)
    # every request: the streaming kernel (direct fp32 distances) must pick the same neighbours and labels as the
    # tensor-core path.  This is a consistency check between two CUDA paths, not oracle parity.
    cache.set_path(fb.FI_PATH_STREAM)
    out2 = cache.lookup_batch(to_device(st.queries))
    torch.cuda.synchronize()
    same_set = (np.sort(out2.topk_idx.cpu().numpy(), 1) == np.sort(got[4], 1)).all(1)
    print(f"config 3: neighbour sets equal on both paths for {int(same_set.sum())} of 8192 requests")
    assert same_set.mean() > 0.99
    np.testing.assert_array_equal(out2.label.cpu().numpy()[same_set], got[0][same_set])
    np.testing.assert_allclose(out2.topk_dist.cpu().numpy()[same_set], got[3][same_set], rtol=1e-5)
    assert 0.3 < got[2].mean() < 0.7
    cache.close()


@pytest.mark.parametrize("batch", [1, 4, 16])
def test_config5_full_latency_shapes(batch):
    w = dg.config5(seed=0, batch=batch)
    st = w.stages[0]
    ref0 = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=1, tau=0.0, rule=fo.RULE_DIST_LE)
    tau = f32(np.percentile(ref0.nd[:, 0], 50.0)) if batch > 1 else f32(ref0.nd[0, 0] * 1.01)
    ref = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=1, tau=tau, rule=fo.RULE_DIST_LE)
    cache = make_cache(st, k=1, num_classes=10, rule=fb.FI_HIT_DIST_LE, tau=tau, max_batch=16)
    out = cache.lookup_batch(to_device(st.queries))
    torch.cuda.synchronize()
    cache.poll_status()
    stats = compare_lookup(out.label.cpu().numpy(), out.conf.cpu().numpy(), out.hit.cpu().numpy(),
                           out.topk_dist.cpu().numpy(), out.topk_idx.cpu().numpy(), ref, storage="bf16", tau=tau,
                           rule=1, cache_labels=st.cache_labels)
    print(stats)
    assert stats.exempt_gap <= 1
    cache.close()
