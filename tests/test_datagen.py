"""The seeded input generators: determinism, shapes and the structure the workloads promise."""
import numpy as np

from paper_2002_02645_b200 import datagen as dg


def test_same_seed_same_bits_and_thread_count_does_not_matter(monkeypatch):
    a = dg.config2(seed=0, shrink=32)
    monkeypatch.setattr(dg, "_workers", lambda: 1)
    b = dg.config2(seed=0, shrink=32)
    c = dg.config2(seed=1, shrink=32)
    for sa, sb, sc in zip(a.stages, b.stages, c.stages):
        assert sa.cache_vecs.dtype == np.uint16
        np.testing.assert_array_equal(sa.cache_vecs, sb.cache_vecs)
        np.testing.assert_array_equal(sa.queries, sb.queries)
        np.testing.assert_array_equal(sa.calib, sb.calib)
        assert (sa.cache_vecs != sc.cache_vecs).any()
    np.testing.assert_array_equal(a.query_classes, b.query_classes)


def test_config1_has_exact_copies_and_relu():
    w = dg.config1(seed=0)
    st = w.stages[0]
    assert st.cache_vecs.shape == (1000, 512) and st.cache_vecs.dtype == np.float32
    assert st.queries.shape == (282, 512)
    assert (st.cache_vecs >= 0).all() and (st.cache_vecs == 0).mean() > 0.2       # ReLU leaves exact zeros
    cp = w.meta["copy_of"]
    assert (cp >= 0).sum() == 26
    for i in np.nonzero(cp >= 0)[0]:
        np.testing.assert_array_equal(st.queries[i], st.cache_vecs[cp[i]])
    assert set(np.unique(st.cache_labels)) == set(range(10))


def test_halfnormal_cascade_class_shift_grows():
    w = dg.config2(seed=0, shrink=32)
    assert [s.dim for s in w.stages] == [2048, 1024, 512, 256]
    sep = []
    for s in w.stages:
        x = dg.stored_to_f64(s.cache_vecs)
        assert (x >= 0).all()
        mu = np.stack([x[s.cache_labels == c].mean(0) for c in range(10)])
        sep.append(np.linalg.norm(mu - mu.mean(0), axis=1).mean() / np.sqrt(s.dim))
    assert sep == sorted(sep)           # separation grows with depth


def test_zipf_class_frequencies():
    p = dg.class_probs(1000, 1.1)
    assert abs(p.sum() - 1.0) < 1e-12 and p[0] / p[9] == np.float64(10.0) ** 1.1
    lab = dg.draw_labels(200000, p, 0, 2)
    counts = np.bincount(lab, minlength=1000)
    assert counts[0] > counts[9] > counts[99] > 0
    assert abs(counts[0] / 200000 - p[0]) < 0.01


def test_latency_workload_shape():
    w = dg.config5(shrink=50, batch=4)
    assert w.stages[0].cache_vecs.shape == (1000, 16384) and w.stages[0].queries.shape == (4, 16384) and w.k == 1
