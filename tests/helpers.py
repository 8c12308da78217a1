"""Shared pieces of the GPU parity tests: moving seeded inputs to the device and the comparison rule.

Comparison rule (CUDA path vs fp64 oracle, same stored bits on both sides)
  - label, hit, compacted miss indices and counts: bit-exact.  The ONE exemption: a query whose oracle k-th /
    (k+1)-th squared-distance gap is below 1e-4 relative (its neighbour set is not decidable in fp32); such
    queries are counted.  In a cascade a request is exempt from the first stage at which its look-up has such a
    gap, onward; before that stage it is compared like every other request.
  - counted as diagnostics, but COMPARED like everything else: queries whose confidence lies within 1e-4 relative
    of the threshold, and queries whose two best label confidences lie within 1e-4 relative of each other.
  - neighbour indices as a set per query; neighbour distances ascending, each within 2e-3 relative (bf16
    storage) or 1e-5 relative (fp32 storage) of the oracle's, and exactly 0 where the oracle has 0.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from paper_2002_02645_b200 import binding as fb

GAP_EXEMPT = 1e-4
NEAR_REL = 1e-4          # diagnostic buckets only: nothing is exempt for being "near"
DIST_TOL = {"bf16": 2e-3, "f32": 1e-5}


def to_device(a: np.ndarray, device="cuda:0") -> torch.Tensor:
    """Stored vectors (float32 or bf16 bit patterns) -> device tensor of the matching torch dtype."""
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.uint16:
        return t.view(torch.int16).to(device).view(torch.bfloat16)
    return t.to(device)


def to_host_tensor(a: np.ndarray, pin: bool = False) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.uint16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.pin_memory() if pin else t


def make_cache(stage, *, k, num_classes, rule=fb.FI_HIT_CONF_GT, metric=fb.FI_METRIC_SQL2, tau=0.0, max_batch=1024,
               path=fb.FI_PATH_AUTO, weights=None, capacity=None, device=0) -> fb.FreezeCache:
    dtype = fb.FI_BF16 if stage.dtype == "bf16" else fb.FI_F32
    n = stage.cache_vecs.shape[0]
    c = fb.FreezeCache(dim=stage.dim, capacity=capacity or max(n, 1), num_classes=num_classes, k=k, dtype=dtype,
                       rule=rule, metric=metric, threshold=float(tau), device=device, max_batch=max_batch, path=path)
    if n > 0:
        w = None if weights is None else torch.from_numpy(np.ascontiguousarray(weights, dtype=np.float32)).to(c.device)
        c.insert(to_device(stage.cache_vecs, c.device), torch.from_numpy(stage.cache_labels).to(c.device), w)
    return c


@dataclass
class ParityStats:
    queries: int = 0
    exempt_gap: int = 0            # the only exemption
    exempt_equal_anyway: int = 0   # exempt queries whose label and hit equal the oracle's all the same
    near_threshold: int = 0        # diagnostics; these queries are compared
    near_label_tie: int = 0
    label_mismatch: int = 0        # outside the exempt bucket
    hit_mismatch: int = 0
    set_mismatch: int = 0
    max_dist_rel_err: float = 0.0

    @property
    def mismatches(self):
        return self.label_mismatch + self.hit_mismatch + self.set_mismatch

    def __str__(self):
        return (f"queries={self.queries} exempt(k-th gap<{GAP_EXEMPT:g})={self.exempt_gap} "
                f"(equal anyway {self.exempt_equal_anyway}) "
                f"near_threshold={self.near_threshold} near_label_tie={self.near_label_tie} "
                f"label_mismatch={self.label_mismatch} hit_mismatch={self.hit_mismatch} "
                f"set_mismatch={self.set_mismatch} max_dist_rel_err={self.max_dist_rel_err:.3g}")


def kth_gap(ora) -> np.ndarray:
    """Relative gap between the k-th and the (k+1)-th squared distance of every query of an oracle result (inf when
    there is no (k+1)-th entry; 0 when both are 0)."""
    b = ora.nd.shape[0]
    k_eff = (ora.ni >= 0).sum(axis=1)
    gap = np.full(b, np.inf)
    for i in range(b):
        if k_eff[i] == 0 or not np.isfinite(ora.next_d[i]):
            continue
        kth = ora.nd[i, k_eff[i] - 1]
        if kth > 0:
            gap[i] = (ora.next_d[i] - kth) / kth
        elif ora.next_d[i] == 0:
            gap[i] = 0.0
    return gap


def _runner_up_gap(nd, lab, w, k_eff, metric):
    """Relative gap between the two largest label confidences of one query (inf when only one label)."""
    conf = {}
    cnt = {}
    for dj, lj, wj in zip(nd[:k_eff], lab[:k_eff], w[:k_eff]):
        dd = np.sqrt(dj) if metric == 1 else dj
        conf[lj] = conf.get(lj, 0.0) + (wj / dd if dd > 0 else np.inf)
        cnt[lj] = cnt.get(lj, 0) + 1
    vals = sorted(((cnt[l] / k_eff) * conf[l] for l in conf), reverse=True)
    if len(vals) < 2 or not np.isfinite(vals[0]):
        return np.inf
    return (vals[0] - vals[1]) / vals[0]


def near_flags(ora, *, tau, rule, metric=0, cache_labels=None, weights=None):
    """Diagnostic buckets of an oracle result: (confidence within NEAR_REL of the threshold, two best label
    confidences within NEAR_REL of each other), one flag per query."""
    b = ora.nd.shape[0]
    near_thr = np.zeros(b, bool)
    near_tie = np.zeros(b, bool)
    for i in range(b):
        k_eff = int((ora.ni[i] >= 0).sum())
        if rule == 0:
            c = ora.conf[i]
            near_thr[i] = bool(np.isfinite(c) and tau > 0 and np.isfinite(tau) and abs(c - tau) / tau < NEAR_REL)
        elif k_eff > 0 and np.isfinite(tau) and tau > 0:
            # distance rule: the winning label's nearest member against the threshold
            idx = ora.ni[i, :k_eff]
            dw = ora.nd[i, :k_eff]
            if cache_labels is not None:
                dw = dw[cache_labels[idx] == ora.label[i]]
            d = np.sqrt(dw[0]) if metric == 1 else dw[0]
            near_thr[i] = abs(d - tau) / tau < NEAR_REL
        if cache_labels is not None and k_eff > 0:
            idx = ora.ni[i, :k_eff]
            w = np.ones(k_eff) if weights is None else np.asarray(weights, dtype=np.float64)[idx]
            near_tie[i] = _runner_up_gap(ora.nd[i], cache_labels[idx], w, k_eff, metric) < NEAR_REL
    return near_thr, near_tie


def compare_lookup(gpu_label, gpu_conf, gpu_hit, gpu_dist, gpu_idx, ora, *, storage, tau, rule, metric=0,
                   cache_labels=None, weights=None, strict=True) -> ParityStats:
    """Element-by-element comparison of one batch; raises AssertionError on a mismatch outside the exempt bucket
    (strict=False counts the mismatches instead)."""
    st = ParityStats()
    b, k = ora.nd.shape
    st.queries = b
    tol = DIST_TOL[storage]
    gaps = kth_gap(ora)
    near_thr, near_tie = near_flags(ora, tau=tau, rule=rule, metric=metric, cache_labels=cache_labels, weights=weights)
    st.near_threshold = int(near_thr.sum())
    st.near_label_tie = int(near_tie.sum())

    def fail(msg):
        if strict:
            raise AssertionError(msg)

    for i in range(b):
        k_eff = int((ora.ni[i] >= 0).sum())
        gap = gaps[i]
        if gap < GAP_EXEMPT:
            st.exempt_gap += 1
            st.exempt_equal_anyway += int(int(gpu_label[i]) == int(ora.label[i]) and int(gpu_hit[i]) == int(ora.hit[i]))
            continue
        where = f"query {i} (gap {gap:.3g}{', near threshold' if near_thr[i] else ''}{', near label tie' if near_tie[i] else ''})"
        if gpu_idx is not None:
            want = set(int(v) for v in ora.ni[i, :k_eff])
            got = set(int(v) for v in gpu_idx[i, :k_eff])
            if want != got:
                st.set_mismatch += 1
                fail(f"{where}: neighbour set {sorted(got)} != {sorted(want)}")
            assert (gpu_idx[i, k_eff:] == -1).all()
        if gpu_dist is not None:
            gd = gpu_dist[i, :k_eff].astype(np.float64)
            assert (np.diff(gd) >= 0).all(), f"{where}: distances not ascending"
            od = ora.nd[i, :k_eff]
            zero = od == 0
            assert (gd[zero] == 0).all(), f"{where}: exact copy must give distance 0"
            if (~zero).any():
                rel = np.abs(gd[~zero] - od[~zero]) / od[~zero]
                st.max_dist_rel_err = max(st.max_dist_rel_err, float(rel.max()))
                assert rel.max() <= tol, f"{where}: distance error {rel.max():.3g} > {tol}"
            assert np.isinf(gpu_dist[i, k_eff:]).all()
        if int(gpu_label[i]) != int(ora.label[i]):
            st.label_mismatch += 1
            fail(f"{where}: label {int(gpu_label[i])} != {int(ora.label[i])}")
        elif np.isinf(ora.conf[i]):
            assert np.isinf(gpu_conf[i]), f"{where}: confidence must be +inf for an exact copy"
        elif ora.conf[i] != 0:
            rel = abs(float(gpu_conf[i]) - ora.conf[i]) / abs(ora.conf[i])
            assert rel <= 5 * tol, f"{where}: confidence error {rel:.3g}"
        if int(gpu_hit[i]) != int(ora.hit[i]):
            st.hit_mismatch += 1
            fail(f"{where}: hit {int(gpu_hit[i])} != {int(ora.hit[i])} "
                 f"(conf {float(gpu_conf[i])!r} vs {ora.conf[i]!r}, tau {tau!r})")
    return st


@dataclass
class CascadeStats:
    requests: int = 0
    exempt: int = 0                # requests with a small k-th gap at some stage of their oracle path
    exempt_equal_anyway: int = 0   # of those: final label and exit stage equal to the oracle's all the same
    near_threshold: int = 0        # look-ups (request, stage) on compared paths; diagnostics only
    near_label_tie: int = 0
    mismatches: int = 0            # compared requests whose label / exit stage / survivor membership differs
    arrivals: tuple = ()

    def __str__(self):
        return (f"requests={self.requests} arrivals={list(self.arrivals)} exempt(k-th gap<{GAP_EXEMPT:g} at some stage)="
                f"{self.exempt} (equal anyway {self.exempt_equal_anyway}) near_threshold={self.near_threshold} "
                f"near_label_tie={self.near_label_tie} mismatches={self.mismatches}")


def compare_cascade(ref, taus, gpu_label, gpu_stage, gpu_conf, gpu_survivors, *, sample_ids=None, stage_labels=None,
                    rule=0, metric=0, conf_rtol=1e-2, strict=True) -> CascadeStats:
    """A cascade on the GPU against the oracle's (`ref`: fi_oracle.CascadeResult over the sampled requests).

    gpu_label / gpu_stage / gpu_conf: per request of the full batch; gpu_survivors[l]: ids alive after stage l.
    sample_ids: the batch ids the oracle ran on (None: the whole batch, in order).
    A request is exempt from the first stage at which its oracle look-up has a k-th/(k+1)-th gap below 1e-4
    relative; before that stage its hit decisions, and hence its membership in every survivor list, must equal the
    oracle's; a request that is never exempt must end with the oracle's label, exit stage and confidence."""
    n = ref.final_label.shape[0]
    n_stage = len(ref.stage_results)
    ids = np.arange(n) if sample_ids is None else np.asarray(sample_ids)
    pos = {int(g): i for i, g in enumerate(ids)}
    st = CascadeStats(requests=n, arrivals=tuple(a.shape[0] for a in ref.active))
    first_exempt = np.full(n, n_stage + 1)       # stage from which a request is exempt (n_stage + 1: never)
    for l, r in enumerate(ref.stage_results):
        act = ref.active[l]
        small = kth_gap(r) < GAP_EXEMPT
        first_exempt[act[small]] = np.minimum(first_exempt[act[small]], l)
        compared = first_exempt[act] > l
        labs = None if stage_labels is None else stage_labels[l]
        nthr, ntie = near_flags(r, tau=taus[l], rule=rule, metric=metric, cache_labels=labs)
        st.near_threshold += int((nthr & compared).sum())
        st.near_label_tie += int((ntie & compared).sum())
    st.exempt = int((first_exempt <= n_stage).sum())

    def fail(msg):
        st.mismatches += 1
        if strict:
            raise AssertionError(msg)

    # survivor lists (miss_idx, miss_count), restricted to the requests still compared after stage l
    for l in range(n_stage):
        got = np.array([pos[int(g)] for g in gpu_survivors[l] if int(g) in pos], dtype=np.int64)
        want = ref.active[l + 1].astype(np.int64)
        got_c, want_c = got[first_exempt[got] > l], want[first_exempt[want] > l]
        if not np.array_equal(got_c, want_c):
            diff = np.setxor1d(got_c, want_c)
            fail(f"stage {l}: survivors differ for compared requests {ids[diff][:8].tolist()}")
        # a request exempt from stage l on must not have been frozen before l
        assert (np.diff(np.asarray(gpu_survivors[l])) > 0).all(), f"stage {l}: survivor ids not ascending"
    lab, stg, cnf = gpu_label[ids], gpu_stage[ids], gpu_conf[ids]
    for i in range(n):
        fe = first_exempt[i]
        if ref.exit_stage[i] < fe:
            # decided before any exemption: everything about the request is fixed
            if int(stg[i]) != int(ref.exit_stage[i]) or int(lab[i]) != int(ref.final_label[i]):
                fail(f"request {int(ids[i])}: (label, stage) ({int(lab[i])}, {int(stg[i])}) != "
                     f"({int(ref.final_label[i])}, {int(ref.exit_stage[i])})")
            elif ref.exit_stage[i] < n_stage and np.isfinite(ref.final_conf[i]):
                assert abs(float(cnf[i]) - ref.final_conf[i]) <= conf_rtol * abs(ref.final_conf[i]), \
                    f"request {int(ids[i])}: confidence {float(cnf[i])!r} vs {ref.final_conf[i]!r}"
        else:
            if int(stg[i]) < fe:
                fail(f"request {int(ids[i])}: frozen at stage {int(stg[i])}, before its first exempt stage {int(fe)}")
            st.exempt_equal_anyway += int(int(stg[i]) == int(ref.exit_stage[i]) and int(lab[i]) == int(ref.final_label[i]))
    return st


def tau_between(values, percentile: float) -> float:
    """A float32 threshold near the given percentile of `values` that no value is close to: the midpoint of two
    neighbouring order statistics at least 1e-3 relative apart.  A threshold taken from the batch's own confidences
    would equal one of them up to rounding, and fp32 cannot decide a comparison whose two sides differ by less than
    its own rounding error (about 1e-7 relative); the tests avoid that construction instead of exempting it."""
    v = np.unique(np.asarray(values, dtype=np.float64)[np.isfinite(values)])
    if v.size == 0:
        return 1.0
    if v.size == 1:
        return f32(v[0] * 0.75)
    i = int(round(percentile / 100.0 * (v.size - 2)))
    order = sorted(range(v.size - 1), key=lambda j: abs(j - i))
    for j in order:
        lo, hi = v[j], v[j + 1]
        if hi - lo > 1e-3 * abs(hi):
            return f32(0.5 * (lo + hi))
    return f32(v[-1] * 1.25)


def f32(x: float) -> float:
    """The float32 value both sides use for a threshold."""
    return float(np.float32(x))
