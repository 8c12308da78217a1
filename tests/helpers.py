"""Shared pieces of the GPU parity tests: moving seeded inputs to the device and the comparison rule.

Comparison rule (CUDA path vs fp64 oracle, same stored bits on both sides)
  - label, hit: bit-exact, except for queries whose oracle k-th / (k+1)-th squared-distance gap is below
    1e-4 relative (the neighbour set itself is then not decidable in fp32); those are counted.
  - also counted, and compared only when decidable: queries whose confidence is within 1e-5 relative of the
    threshold, or whose two best label confidences are within 1e-5 relative of each other (the GPU forms the
    confidence in fp32, the oracle in fp64).
  - neighbour indices as a set per query; neighbour distances ascending, each within 2e-3 relative (bf16
    storage) or 1e-5 relative (fp32 storage) of the oracle's, and exactly 0 where the oracle has 0.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from paper_2002_02645_b200 import binding as fb

GAP_EXEMPT = 1e-4
NEAR_REL = 1e-5
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
    exempt_gap: int = 0
    near_threshold: int = 0
    near_label_tie: int = 0
    label_mismatch: int = 0
    hit_mismatch: int = 0
    set_mismatch: int = 0
    max_dist_rel_err: float = 0.0

    def __str__(self):
        return (f"queries={self.queries} exempt(k-th gap<{GAP_EXEMPT:g})={self.exempt_gap} "
                f"near_threshold={self.near_threshold} near_label_tie={self.near_label_tie} "
                f"label_mismatch={self.label_mismatch} hit_mismatch={self.hit_mismatch} "
                f"set_mismatch={self.set_mismatch} max_dist_rel_err={self.max_dist_rel_err:.3g}")


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


def compare_lookup(gpu_label, gpu_conf, gpu_hit, gpu_dist, gpu_idx, ora, *, storage, tau, rule, metric=0,
                   cache_labels=None, weights=None, strict=True) -> ParityStats:
    """Element-by-element comparison of one batch; raises AssertionError on a mismatch that is not exempt."""
    st = ParityStats()
    b, k = ora.nd.shape
    st.queries = b
    tol = DIST_TOL[storage]
    for i in range(b):
        k_eff = int((ora.ni[i] >= 0).sum())
        kth = ora.nd[i, k_eff - 1] if k_eff > 0 else 0.0
        gap = (ora.next_d[i] - kth) / kth if (k_eff > 0 and np.isfinite(ora.next_d[i]) and kth > 0) else np.inf
        if k_eff > 0 and np.isfinite(ora.next_d[i]) and kth == 0 and ora.next_d[i] == 0:
            gap = 0.0
        exempt = gap < GAP_EXEMPT
        st.exempt_gap += int(exempt)
        if gpu_idx is not None and not exempt:
            want = set(int(v) for v in ora.ni[i, :k_eff])
            got = set(int(v) for v in gpu_idx[i, :k_eff])
            if want != got:
                st.set_mismatch += 1
                if strict:
                    raise AssertionError(f"query {i}: neighbour set {sorted(got)} != {sorted(want)} (gap {gap:.3g})")
            assert (gpu_idx[i, k_eff:] == -1).all()
        if gpu_dist is not None and not exempt:
            gd = gpu_dist[i, :k_eff].astype(np.float64)
            assert (np.diff(gd) >= 0).all(), f"query {i}: distances not ascending"
            od = ora.nd[i, :k_eff]
            zero = od == 0
            assert (gd[zero] == 0).all(), f"query {i}: exact copy must give distance 0"
            if (~zero).any():
                rel = np.abs(gd[~zero] - od[~zero]) / od[~zero]
                st.max_dist_rel_err = max(st.max_dist_rel_err, float(rel.max()))
                assert rel.max() <= tol, f"query {i}: distance error {rel.max():.3g} > {tol}"
            assert np.isinf(gpu_dist[i, k_eff:]).all()
        # decidability of the vote and of the threshold test in fp32
        near_tie = False
        if cache_labels is not None and k_eff > 0:
            idx = ora.ni[i, :k_eff]
            w = np.ones(k_eff) if weights is None else np.asarray(weights, dtype=np.float64)[idx]
            near_tie = _runner_up_gap(ora.nd[i], cache_labels[idx], w, k_eff, metric) < NEAR_REL
        st.near_label_tie += int(near_tie)
        if rule == 0:
            c = ora.conf[i]
            near_thr = np.isfinite(c) and tau > 0 and abs(c - tau) / tau < NEAR_REL
        else:
            near_thr = False
        st.near_threshold += int(near_thr)
        if not exempt and not near_tie:
            if int(gpu_label[i]) != int(ora.label[i]):
                st.label_mismatch += 1
                if strict:
                    raise AssertionError(f"query {i}: label {int(gpu_label[i])} != {int(ora.label[i])}")
            if np.isinf(ora.conf[i]):
                assert np.isinf(gpu_conf[i]), f"query {i}: confidence must be +inf for an exact copy"
            elif ora.conf[i] != 0:
                rel = abs(float(gpu_conf[i]) - ora.conf[i]) / abs(ora.conf[i])
                assert rel <= 5 * tol, f"query {i}: confidence error {rel:.3g}"
            if not near_thr and int(gpu_hit[i]) != int(ora.hit[i]):
                st.hit_mismatch += 1
                if strict:
                    raise AssertionError(f"query {i}: hit {int(gpu_hit[i])} != {int(ora.hit[i])} "
                                         f"(conf {float(gpu_conf[i])!r} vs {ora.conf[i]!r}, tau {tau!r})")
    return st


def f32(x: float) -> float:
    """The float32 value both sides use for a threshold."""
    return float(np.float32(x))
