"""Pins for the fp64 CPU oracle: everything here is fixed by the paper's formulas or by mathematics,
never by the oracle itself (and never by the CUDA path)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import fi_oracle as fo
from paper_2002_02645_b200 import datagen as dg

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ independent brute force (numpy only)

def brute_neighbours(q, x, k):
    """Full sort of all N distances under (D, n); independent of the oracle's selection code."""
    D = ((q[:, None, :].astype(np.float64) - x[None, :, :].astype(np.float64)) ** 2).sum(-1)
    order = np.stack([np.lexsort((np.arange(x.shape[0]), D[b])) for b in range(q.shape[0])])
    kk = min(k, x.shape[0])
    return D, order[:, :kk]


def brute_vote(d, lab, w, k_eff, metric=0):
    """Dictionary-based restatement of Sec. 3's heuristic for cross-checking on random small cases."""
    score, count, first = {}, {}, {}
    for rank, (dj, lj, wj) in enumerate(zip(d, lab, w)):
        dd = np.sqrt(dj) if metric == 1 else dj
        score[lj] = score.get(lj, 0.0) + (wj / dd if dd > 0 else np.inf)
        count[lj] = count.get(lj, 0) + 1
        first.setdefault(lj, rank)
    conf = {l: (count[l] / k_eff) * score[l] for l in score}
    best = sorted(conf, key=lambda l: (-conf[l], -count[l], first[l]))[0]
    return best, conf[best]


# ------------------------------------------------------------------ P3 / golden: hand-evaluated votes

def _golden_votes():
    rows = []
    with open(os.path.join(GOLDEN, "vote_hand_case.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, tuples, label, conf = [s.strip() for s in line.split("|")]
            pairs = [t.split(":") for t in tuples.split()]
            rows.append((int(k), [int(p[0]) for p in pairs], [float(p[1]) for p in pairs], int(label),
                         float(Fraction(conf))))
    return rows


@pytest.mark.parametrize("k,labels,dists,want_label,want_conf", _golden_votes())
def test_vote_hand_cases(k, labels, dists, want_label, want_conf):
    assert len(labels) == k
    label, conf, _ = fo.vote(dists, labels, tau=0.0)
    assert label == want_label
    assert conf == pytest.approx(want_conf, rel=1e-15)


def test_vote_is_not_plain_majority():
    # Sec. 3: closeness counts, so one very close neighbour can outvote two far ones
    label, conf, _ = fo.vote([0.25, 1.0, 2.0], [1, 0, 0])
    assert label == 1 and conf == pytest.approx(4.0 / 3.0)


# ------------------------------------------------------------------ P1 / P2: closed forms

def test_k1_closed_form_and_kmeans_rule():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(50, 7)).astype(np.float32)
    q = rng.normal(size=(9, 7)).astype(np.float32)
    lab = rng.integers(0, 4, 50).astype(np.int32)
    frac = rng.uniform(0.3, 1.0, 50).astype(np.float32)
    D, order = brute_neighbours(q, x, 1)
    r = fo.lookup(q, x, lab, k=1, tau=0.0)
    np.testing.assert_array_equal(r.ni[:, 0], order[:, 0])
    np.testing.assert_array_equal(r.label, lab[order[:, 0]])
    np.testing.assert_allclose(r.conf, 1.0 / D[np.arange(9), order[:, 0]], rtol=1e-14)
    # Sec. 4: k-means entry <centre, majority label, fraction f> -> confidence f / distance
    rw = fo.lookup(q, x, lab, k=1, tau=0.0, weights=frac)
    np.testing.assert_allclose(rw.conf, frac[order[:, 0]].astype(np.float64) / D[np.arange(9), order[:, 0]], rtol=1e-14)
    np.testing.assert_array_equal(rw.label, r.label)


def test_equal_distance_same_label_closed_form():
    # k cache points on a sphere of squared radius 4 around the query, same label: conf = k / d
    k = 6
    dirs = np.eye(k, dtype=np.float32) * 2.0
    far = np.full((3, k), 50.0, dtype=np.float32)
    x = np.concatenate([dirs, far])
    lab = np.array([2] * k + [5, 5, 5], dtype=np.int32)
    q = np.zeros((1, k), dtype=np.float32)
    r = fo.lookup(q, x, lab, k=k, tau=1.0)
    assert r.label[0] == 2 and r.conf[0] == pytest.approx(k / 4.0, rel=1e-15) and r.hit[0] == 1
    r2 = fo.lookup(q, x, lab, k=k, tau=1.0, metric=fo.METRIC_L2)
    assert r2.conf[0] == pytest.approx(k / 2.0, rel=1e-15)


# ------------------------------------------------------------------ P4: brute force on tiny integer inputs

@pytest.mark.parametrize("seed", range(12))
def test_brute_force_integer_coordinates(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 9))
    d = int(rng.integers(1, 4))
    b = int(rng.integers(1, 6))
    k = int(rng.integers(1, 6))
    x = rng.integers(-3, 4, size=(n, d)).astype(np.float32)     # many exact ties
    q = rng.integers(-3, 4, size=(b, d)).astype(np.float32) + np.float32(0.5)   # never d = 0
    lab = rng.integers(0, 3, n).astype(np.int32)
    w = rng.uniform(0.5, 1.0, n).astype(np.float32)
    D, order = brute_neighbours(q, x, k)
    r = fo.lookup(q, x, lab, k=k, tau=0.37, weights=w)
    k_eff = min(k, n)
    for i in range(b):
        np.testing.assert_array_equal(r.ni[i, :k_eff], order[i])
        assert (r.ni[i, k_eff:] == -1).all() and np.isinf(r.nd[i, k_eff:]).all()
        np.testing.assert_array_equal(r.nd[i, :k_eff], D[i, order[i]])      # integers + .5: exact
        bl, bc = brute_vote(D[i, order[i]], lab[order[i]], w[order[i]].astype(np.float64), k_eff)
        assert r.label[i] == bl
        assert r.conf[i] == pytest.approx(bc, rel=1e-14)
        assert r.hit[i] == (bc > 0.37)
    # (k+1)-th distance
    full = np.sort(D, axis=1)
    for i in range(b):
        want = full[i, k] if n > k else np.inf
        assert r.next_d[i] == want


def test_distance_matrix_orientation_and_terms():
    # asymmetric shapes catch a transposed operand; a dropped or mis-signed term fails the identity
    x = np.array([[0, 0, 0], [1, 2, 3], [4, 0, -1], [2, 2, 2]], dtype=np.float32)
    q = np.array([[1, 1, 1], [0, -2, 5]], dtype=np.float32)
    D = fo.sqdist(q, x)
    want = np.array([[3, 0 + 1 + 4, 9 + 1 + 4, 3], [29, 1 + 16 + 4, 16 + 4 + 36, 4 + 16 + 9]], dtype=np.float64)
    np.testing.assert_array_equal(D, want)


def test_bf16_values_are_decoded_exactly():
    rng = np.random.default_rng(5)
    xf = rng.normal(size=(20, 33)).astype(np.float32)
    qf = rng.normal(size=(4, 33)).astype(np.float32)
    xb, qb = dg.f32_to_bf16_bits(xf), dg.f32_to_bf16_bits(qf)
    # round-to-nearest-even reference: the bf16 value is within half a bf16 ulp and has 8 significant bits
    dec = dg.bf16_bits_to_f32(xb)
    assert (np.abs(dec - xf) <= np.abs(xf) * 2.0 ** -8).all()
    assert ((dec.view(np.uint32) & 0xFFFF) == 0).all()
    D = fo.sqdist(qb, xb)
    want = ((dg.stored_to_f64(qb)[:, None, :] - dg.stored_to_f64(xb)[None, :, :]) ** 2).sum(-1)
    np.testing.assert_allclose(D, want, rtol=1e-14)


def test_bf16_rounding_ties_to_even():
    # 1 + 2^-8 lies exactly between two bf16 values: ties go to the even mantissa (1.0);
    # 1 + 3*2^-8 ties up to 1 + 2^-6
    v = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20], dtype=np.float32)
    got = dg.bf16_bits_to_f32(dg.f32_to_bf16_bits(v))
    np.testing.assert_array_equal(got, np.array([1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7], dtype=np.float32))


# ------------------------------------------------------------------ P7: textbook cross-check through another formula

def test_against_expanded_form_numpy():
    rng = np.random.default_rng(7)
    x = rng.normal(size=(300, 40))
    q = rng.normal(size=(17, 40))
    xf, qf = x.astype(np.float32), q.astype(np.float32)
    lab = rng.integers(0, 5, 300).astype(np.int32)
    x64, q64 = xf.astype(np.float64), qf.astype(np.float64)
    E = (q64 ** 2).sum(1)[:, None] + (x64 ** 2).sum(1)[None, :] - 2.0 * q64 @ x64.T     # ||q||^2+||c||^2-2q.c
    r = fo.lookup(qf, xf, lab, k=4, tau=0.0)
    np.testing.assert_array_equal(r.ni, np.argsort(E, axis=1, kind="stable")[:, :4])
    np.testing.assert_allclose(r.nd, np.sort(E, axis=1)[:, :4], rtol=1e-10)
    r1 = fo.lookup(qf, xf, lab, k=1, tau=0.0)
    np.testing.assert_array_equal(r1.label, lab[np.argmin(E, axis=1)])


# ------------------------------------------------------------------ P5: invariants

def _small_case(seed=3, n=200, d=16, b=24, c=4):
    rng = np.random.default_rng(seed)
    x = rng.normal(size=(n, d)).astype(np.float32)
    q = rng.normal(size=(b, d)).astype(np.float32)
    lab = rng.integers(0, c, n).astype(np.int32)
    return x, q, lab


def test_identical_query_hits_with_distance_zero():
    # observation O1 (Sec. 2): an identical intermediate output must give the same label
    x, q, lab = _small_case()
    q[:5] = x[[7, 3, 199, 0, 50]]
    for k in (1, 3):
        r = fo.lookup(q, x, lab, k=k, tau=1e30)
        np.testing.assert_array_equal(r.ni[:5, 0], [7, 3, 199, 0, 50])
        assert (r.nd[:5, 0] == 0.0).all() and np.isinf(r.conf[:5]).all() and (r.hit[:5] == 1).all()
        np.testing.assert_array_equal(r.label[:5], lab[[7, 3, 199, 0, 50]])
        assert (r.hit[5:] == 0).all()
    rd = fo.lookup(q, x, lab, k=1, tau=0.0, rule=fo.RULE_DIST_LE)
    assert (rd.hit[:5] == 1).all() and (rd.hit[5:] == 0).all()


def test_hit_count_monotone_in_threshold_and_labels_independent():
    # Sec. 4: raising the threshold lowers the share of points frozen
    x, q, lab = _small_case(b=64)
    taus = [0.0, 0.01, 0.05, 0.1, 0.2, 0.5, 1.0, 10.0]
    base = fo.lookup(q, x, lab, k=5, tau=taus[0])
    hits = []
    for t in taus:
        r = fo.lookup(q, x, lab, k=5, tau=t)
        np.testing.assert_array_equal(r.label, base.label)
        np.testing.assert_array_equal(r.ni, base.ni)
        np.testing.assert_array_equal(r.hit, (r.conf > t).astype(np.uint8))      # strict
        hits.append(int(r.hit.sum()))
    assert hits == sorted(hits, reverse=True) and hits[0] == 64 and hits[-1] == 0
    hd = [int(fo.lookup(q, x, lab, k=5, tau=t, rule=fo.RULE_DIST_LE).hit.sum()) for t in [0, 5, 10, 20, 40, 1e9]]
    assert hd == sorted(hd) and hd[0] == 0 and hd[-1] == 64


def test_strict_threshold_at_equality():
    x = np.array([[2.0, 0.0]], dtype=np.float32)
    q = np.zeros((1, 2), dtype=np.float32)
    lab = np.array([1], dtype=np.int32)
    assert fo.lookup(q, x, lab, k=1, tau=0.25).hit[0] == 0          # conf == tau: not a hit (">" in Pseudocode 1)
    assert fo.lookup(q, x, lab, k=1, tau=np.nextafter(0.25, 0)).hit[0] == 1
    assert fo.lookup(q, x, lab, k=1, tau=4.0, rule=fo.RULE_DIST_LE).hit[0] == 1     # "<=" is inclusive
    assert fo.lookup(q, x, lab, k=1, tau=np.nextafter(4.0, 0), rule=fo.RULE_DIST_LE).hit[0] == 0


def test_scaling_translation_permutation_append():
    x, q, lab = _small_case()
    r = fo.lookup(q, x, lab, k=5, tau=0.0)
    s = np.float32(4.0)                                              # power of two: exact in fp32
    rs = fo.lookup(q * s, x * s, lab, k=5, tau=0.0)
    np.testing.assert_array_equal(rs.ni, r.ni)
    np.testing.assert_allclose(rs.nd, r.nd * 16.0, rtol=1e-15)
    np.testing.assert_allclose(rs.conf, r.conf / 16.0, rtol=1e-15)
    # translation by integers on integer-valued inputs is exact
    xi, qi = np.round(x * 8), np.round(q * 8) + np.float32(0.5)
    ri = fo.lookup(qi, xi, lab, k=5, tau=0.0)
    rt = fo.lookup(qi + 100, xi + 100, lab, k=5, tau=0.0)
    np.testing.assert_array_equal(rt.ni, ri.ni)
    np.testing.assert_array_equal(rt.nd, ri.nd)
    # permuting the cache rows permutes indices only
    perm = np.random.default_rng(9).permutation(x.shape[0])
    rp = fo.lookup(q, x[perm], lab[perm], k=5, tau=0.0)
    np.testing.assert_array_equal(perm[rp.ni], r.ni)
    np.testing.assert_array_equal(rp.label, r.label)
    np.testing.assert_allclose(rp.conf, r.conf, rtol=1e-15)
    # rows farther than every current k-th neighbour change nothing
    far = np.full((10, x.shape[1]), 1e3, dtype=np.float32)
    ra = fo.lookup(q, np.concatenate([x, far]), np.concatenate([lab, np.zeros(10, np.int32)]), k=5, tau=0.0)
    np.testing.assert_array_equal(ra.ni, r.ni)
    np.testing.assert_array_equal(ra.conf, r.conf)


def test_l2_metric_takes_square_root_of_winners():
    x, q, lab = _small_case()
    r0 = fo.lookup(q, x, lab, k=3, tau=0.0)
    r1 = fo.lookup(q, x, lab, k=3, tau=0.0, metric=fo.METRIC_L2)
    np.testing.assert_array_equal(r0.ni, r1.ni)
    for i in range(q.shape[0]):
        bl, bc = brute_vote(r0.nd[i], lab[r0.ni[i]], np.ones(3), 3, metric=1)
        assert r1.label[i] == bl and r1.conf[i] == pytest.approx(bc, rel=1e-14)


def test_k_larger_than_cache_and_empty_cache():
    x = np.array([[0.0, 1.0], [0.0, 3.0]], dtype=np.float32)
    lab = np.array([4, 4], dtype=np.int32)
    q = np.zeros((1, 2), dtype=np.float32)
    r = fo.lookup(q, x, lab, k=5, tau=0.0)
    # k_eff = 2: S = 2/2, sum = 1/1 + 1/9
    assert r.label[0] == 4 and r.conf[0] == pytest.approx(1.0 + 1.0 / 9.0, rel=1e-15)
    assert list(r.ni[0]) == [0, 1, -1, -1, -1] and np.isinf(r.next_d[0])
    e = fo.lookup(q, np.zeros((0, 2), np.float32), np.zeros(0, np.int32), k=3, tau=0.0)
    assert e.label[0] == -1 and e.conf[0] == 0.0 and e.hit[0] == 0


def test_vote_tie_breaks():
    # equal confidence, different counts: (2/4)(1/1+1/1) = 1 vs (1/4)(1/0.25) = 1 -> larger m wins
    label, conf, _ = fo.vote([0.25, 1.0, 1.0, 9.0], [8, 3, 3, 6])
    assert conf == 1.0 and label == 3
    # equal confidence and count: the label whose nearest member comes first
    label, _, _ = fo.vote([2.0, 2.0], [6, 1])
    assert label == 6
    # +inf == +inf: two exact copies with different labels -> first under (D, n)
    label, conf, hit = fo.vote([0.0, 0.0, 1.0], [9, 2, 2], tau=1e300)
    assert np.isinf(conf) and hit and label == 2        # m = 2 beats m = 1 at equal (infinite) confidence


# ------------------------------------------------------------------ P8: the two hit rules for k = 1

def test_hit_rules_agree_for_k1():
    x, q, lab = _small_case(b=80)
    tau_d = 17.3
    a = fo.lookup(q, x, lab, k=1, tau=tau_d, rule=fo.RULE_DIST_LE)
    b = fo.lookup(q, x, lab, k=1, tau=1.0 / tau_d, rule=fo.RULE_CONF_GT)
    assert 0 < a.hit.sum() < 80
    np.testing.assert_array_equal(a.hit, b.hit)


# ------------------------------------------------------------------ P6: compaction and cascade

def test_compaction_invariants():
    rng = np.random.default_rng(11)
    active = np.sort(rng.choice(1000, 300, replace=False)).astype(np.int32)
    hit = (rng.random(300) < 0.4).astype(np.uint8)
    miss = fo.compact(active, hit)
    assert miss.shape[0] == 300 - hit.sum()
    assert (np.diff(miss) > 0).all()
    np.testing.assert_array_equal(miss, active[hit == 0])
    assert fo.compact(active, np.ones(300, np.uint8)).shape[0] == 0
    np.testing.assert_array_equal(fo.compact(active, np.zeros(300, np.uint8)), active)
    assert fo.compact(np.zeros(0, np.int32), np.zeros(0, np.uint8)).shape[0] == 0


def test_cascade_partition_and_limits():
    w = dg.config2(seed=0, shrink=64)
    sq = [s.queries for s in w.stages]
    sc = [s.cache_vecs for s in w.stages]
    sl = [s.cache_labels for s in w.stages]
    b0 = sq[0].shape[0]
    # thresholds from the calibration draws, so that every stage freezes some and passes some
    taus = []
    for s, p in zip(w.stages, w.meta["percentiles"]):
        c = fo.lookup(s.calib, s.cache_vecs, s.cache_labels, k=w.k, tau=0.0).conf
        taus.append(float(np.percentile(c, p)))
    r = fo.cascade(sq, sc, sl, taus, k=w.k)
    # frozen sets of all stages and the survivors partition the batch
    assert r.active[0].shape[0] == b0
    frozen_total = 0
    for l in range(4):
        ids, nxt = r.active[l], r.active[l + 1]
        assert (np.diff(ids) > 0).all() if ids.size > 1 else True
        froze = np.setdiff1d(ids, nxt)
        assert (r.exit_stage[froze] == l).all()
        assert nxt.shape[0] == ids.shape[0] - int(r.stage_results[l].hit.sum())
        frozen_total += froze.shape[0]
    assert frozen_total + r.active[4].shape[0] == b0
    assert (r.exit_stage[r.active[4]] == 4).all() and (r.final_label[r.active[4]] == -1).all()
    assert 0 < frozen_total
    # a request frozen at stage l carries stage l's look-up result computed on its own row
    for l in range(4):
        ids = r.active[l]
        solo = fo.lookup(sq[l][ids], sc[l], sl[l], k=w.k, tau=taus[l])
        np.testing.assert_array_equal(solo.label, r.stage_results[l].label)
        np.testing.assert_array_equal(solo.hit, r.stage_results[l].hit)
    # tau = +inf: nobody freezes; tau = 0: everybody with a finite distance freezes at stage 0
    r_inf = fo.cascade(sq, sc, sl, [np.inf] * 4, k=w.k)
    assert (r_inf.exit_stage == 4).all() and r_inf.active[4].shape[0] == b0
    r_0 = fo.cascade(sq, sc, sl, [0.0] * 4, k=w.k)
    assert (r_0.exit_stage == 0).all() and all(a.shape[0] == 0 for a in r_0.active[1:])


# ------------------------------------------------------------------ workload shapes (Table 1)

def test_table1_memory_arithmetic():
    vals = {}
    with open(os.path.join(GOLDEN, "table1_memory.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                key, v = line.split()
                vals[key] = float(v)
    per_image = 2 * (64 * 32 * 32 + 128 * 16 * 16 + 256 * 8 * 8 + 512 * 4 * 4)
    mib = 1024.0 * 1024.0
    assert vals["entries_per_layer"] * per_image * 4 / mib == vals["knn_raw_mb"]
    assert vals["blocks"] * vals["entries_per_layer"] * vals["reduced_dim"] * 8 / mib == vals["knn_reduced_mb"]
    assert vals["blocks"] * vals["clusters"] * vals["reduced_dim"] * 8 / mib == vals["kmeans_reduced_mb"]
    # the four-stage cascade workload uses exactly these activation sizes
    w = dg.config2(shrink=64)
    assert [s.dim * 64 for s in w.stages] == [64 * 32 * 32, 128 * 16 * 16, 256 * 8 * 8, 512 * 4 * 4]


# ------------------------------------------------------------------ ComputeThresholds (Pseudocode 1, Sec. 3.1 (ii))

def test_compute_threshold_hand_case_and_zero_error_property():
    # three cached points on a line, labels 0 / 1 / 1; k = 1 so conf = 1 / squared distance
    x = np.array([[0.0], [10.0], [20.0]], dtype=np.float32)
    lab = np.array([0, 1, 1], dtype=np.int32)
    v = np.array([[1.0], [9.5], [4.0], [12.0]], dtype=np.float32)         # nearest: 0, 1, 0, 1
    model = np.array([0, 0, 1, 1], dtype=np.int32)                         # items 1 and 2 are looked up wrongly
    tau, wrong = fo.compute_threshold(v, x, lab, model, k=1)
    assert wrong == 2 and tau == max(1.0 / 0.25, 1.0 / 16.0)               # confidences 4 and 1/16
    assert fo.compute_threshold(v[[0, 3]], x, lab, model[[0, 3]], k=1) == (0.0, 0)   # nothing wrong: stays at 0
    # "zero error on the validation data": with that threshold every validation hit carries the model's label,
    # and more validation items can only raise it
    xs, qs, labs = _small_case(seed=13, n=300, b=120, c=5)
    rng = np.random.default_rng(14)
    model = np.where(rng.random(120) < 0.8, fo.lookup(qs, xs, labs, k=3, tau=0.0).label, 4).astype(np.int32)
    tau, wrong = fo.compute_threshold(qs, xs, labs, model, k=3)
    r = fo.lookup(qs, xs, labs, k=3, tau=tau)
    assert wrong > 0 and (r.label[r.hit == 1] == model[r.hit == 1]).all()
    assert tau == r.conf[r.label != model].max()
    tau_half, _ = fo.compute_threshold(qs[:60], xs, labs, model[:60], k=3)
    assert tau_half <= tau


# ------------------------------------------------------------------ k-means cache construction (Sec. 2.1, Sec. 4)

def test_kmeans_step_hand_case_ties_and_empty_cluster():
    pts = np.array([[0.0], [1.0], [2.0], [10.0], [11.0], [5.5]], dtype=np.float32)
    lab = np.array([3, 3, 1, 2, 2, 1], dtype=np.int32)
    cen = np.array([[1.0], [10.0], [100.0]], dtype=np.float32)
    s = fo.kmeans_step(pts, cen, lab, num_classes=4)
    # 5.5 is equally far from 1 and 10: ties go to the smaller centre index
    assert list(s.assign) == [0, 0, 0, 1, 1, 0]
    np.testing.assert_allclose(s.centres[:, 0], [(0 + 1 + 2 + 5.5) / 4, 10.5, 100.0])     # the empty cluster keeps its centre
    assert list(s.counts) == [4, 2, 0]
    # cluster 0 holds labels 3, 3, 1, 1: a tie, the smaller label wins with share 2/4
    assert list(s.majority) == [1, 2, -1] and list(s.fraction) == [0.5, 1.0, 0.0]


def test_kmeans_step_against_sklearn_and_invariants():
    from sklearn.cluster import KMeans
    rng = np.random.default_rng(21)
    true = rng.normal(size=(6, 12)) * 4
    lab = rng.integers(0, 6, 900).astype(np.int32)
    pts = (true[lab] + rng.normal(size=(900, 12))).astype(np.float32)
    init = pts[rng.choice(900, 6, replace=False)].copy()
    s = fo.kmeans_step(pts, init, lab, num_classes=6)
    km = KMeans(n_clusters=6, init=init.astype(np.float64), n_init=1, max_iter=1, tol=0.0, algorithm="lloyd").fit(
        pts.astype(np.float64))
    np.testing.assert_allclose(s.centres, km.cluster_centers_, rtol=1e-9, atol=1e-9)
    assert s.counts.sum() == 900
    np.testing.assert_allclose((s.centres * s.counts[:, None]).sum(0) / 900, pts.astype(np.float64).mean(0), rtol=1e-12)
    # Lloyd iterations never increase the within-cluster sum of squares
    cen, inertia = init, []
    for _ in range(4):
        st = fo.kmeans_step(pts, cen, lab, num_classes=6)
        inertia.append(((pts.astype(np.float64) - cen.astype(np.float64)[st.assign]) ** 2).sum())
        cen = st.centres.astype(np.float32)
    assert all(a >= b * (1 - 1e-6) for a, b in zip(inertia, inertia[1:]))
    # the majority share of a non-empty cluster lies in [1/classes, 1]; clusters that caught a single blob are pure
    # (Sec. 2.1's observation on cluster purity)
    live = st.counts > 0
    assert (st.fraction[live] >= 1.0 / 6).all() and (st.fraction[live] <= 1.0).all() and (st.fraction[live] > 0.95).any()


# ------------------------------------------------------------------ cache rows split into shards

def test_merge_of_row_shards_equals_the_unsharded_lookup():
    x, q, lab = _small_case(seed=23, n=301, b=40, c=5)
    w = np.random.default_rng(24).uniform(0.5, 1.0, 301).astype(np.float32)
    whole = fo.lookup(q, x, lab, k=4, tau=0.03, weights=w)
    cuts = [0, 100, 101, 250, 301]                                    # uneven shards, one of a single row
    parts = [fo.lookup(q, x[a:b], lab[a:b], k=4, tau=0.03, weights=w[a:b]) for a, b in zip(cuts, cuts[1:])]
    merged = fo.merge_shards(parts, cuts[:-1], [lab[a:b] for a, b in zip(cuts, cuts[1:])], k=4, tau=0.03,
                             shard_weights=[w[a:b] for a, b in zip(cuts, cuts[1:])])
    np.testing.assert_array_equal(merged.ni, whole.ni)
    np.testing.assert_array_equal(merged.nd, whole.nd)
    np.testing.assert_array_equal(merged.label, whole.label)
    np.testing.assert_array_equal(merged.conf, whole.conf)
    np.testing.assert_array_equal(merged.hit, whole.hit)


# ------------------------------------------------------------------ projection in front of the look-up (Sec. 3)

def test_bf16_rounding_against_the_library_conversion_and_hand_ties():
    import torch
    rng = np.random.default_rng(5)
    x32 = (rng.standard_normal(100000) * 10.0 ** rng.uniform(-40, 38, 100000)).astype(np.float32)
    x32 = np.concatenate([x32, np.array([0.0, -0.0, 1e-45, 1e-40, 3.38e38, 3.4e38, np.inf, -np.inf], np.float32)])
    want = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(fo.round_to_bf16_bits(x32.astype(np.float64)), want)   # float32 inputs: one rounding
    # ties by hand: bf16 keeps 8 significand bits, so 1 + 2^-8 lies half-way between 1 and 1 + 2^-7
    one, step = 0x3F80, 2.0 ** -7
    assert fo.round_to_bf16_bits(np.array([1 + step / 2]))[0] == one            # tie -> even (1.0)
    assert fo.round_to_bf16_bits(np.array([1 + 3 * step / 2]))[0] == one + 2    # tie -> even (1 + 2 steps)
    assert fo.round_to_bf16_bits(np.array([1 + step / 2 + 1e-12]))[0] == one + 1
    # a float64 value just above a tie must round up even though float32 would first land on the tie
    assert fo.round_to_bf16_bits(np.array([1 + step / 2 + 2.0 ** -40]))[0] == one + 1
    np.testing.assert_array_equal(fo.bf16_bits_to_f64(np.array([one, one + 1], np.uint16)), [1.0, 1 + step])


def test_projection_hand_case_identity_and_bias():
    w = np.array([[1.0, 2.0, -1.0, 0.0], [0.5, 0.0, 0.0, 4.0]], np.float32)
    x = np.array([[0.5, 0.25, 3.0, 1.0], [2.0, 1.0, 0.0, -1.0]], np.float32)
    b = np.array([0.125, -1.0], np.float32)
    bits, pre, mag = fo.project(x, w, b)
    np.testing.assert_array_equal(pre, [[-1.875, 3.25], [4.125, -4.0]])          # by hand
    np.testing.assert_array_equal(mag, [[4.125, 5.25], [4.125, 6.0]])
    np.testing.assert_array_equal(fo.bf16_bits_to_f64(bits), [[0.0, 3.25], [4.125, 0.0]])
    # identity weights: the projection is the rectifier; bf16 inputs come back bit for bit
    rng = np.random.default_rng(6)
    xb = fo.round_to_bf16_bits(rng.standard_normal((5, 16)))
    eye = fo.round_to_bf16_bits(np.eye(16))
    got, _, _ = fo.project(xb, eye)
    want = np.where(fo.bf16_bits_to_f64(xb) > 0, xb, 0).astype(np.uint16)
    np.testing.assert_array_equal(got, want)
    # operands are not transposed: a non-square W [out=3, in=16] gives 3 outputs per row
    w3 = fo.round_to_bf16_bits(rng.standard_normal((3, 16)))
    got3, pre3, _ = fo.project(xb, w3)
    assert got3.shape == (5, 3)
    np.testing.assert_allclose(pre3[2, 1], float(fo.bf16_bits_to_f64(xb[2]) @ fo.bf16_bits_to_f64(w3[1])), rtol=1e-15)
