"""ctypes front end of the fp64 CPU oracle (`fi_oracle.c`) plus the cascade driver.

TEST INFRASTRUCTURE ONLY.  Imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg; never by the product path.  Shares no code with
the CUDA path.  See the header of `fi_oracle.c` for what is computed and which
passages of the paper each step follows.

`cascade()` follows Pseudocode 1 (FreezeInference): stage l looks up only the
requests that no earlier stage froze; a hit records (label, confidence, stage);
requests that survive every stage keep label -1 and exit_stage = number of
stages, standing for "the model's own output layer answers".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fi_oracle.c")
_LIB = os.path.join(_HERE, "libfi_oracle.so")

METRIC_SQL2, METRIC_L2 = 0, 1
RULE_CONF_GT, RULE_DIST_LE = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2 plus OpenMP; no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-ftree-vectorize", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        vp, i64, i32, dbl = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_double
        _lib.fio_sqdist.argtypes = [vp, vp, i32, i64, i64, i64, vp]
        _lib.fio_sqdist.restype = None
        _lib.fio_select.argtypes = [vp, i64, i32, vp, vp]
        _lib.fio_select.restype = None
        _lib.fio_vote.argtypes = [vp, vp, vp, i32, i32, i32, dbl, vp, vp, vp]
        _lib.fio_vote.restype = None
        _lib.fio_lookup.argtypes = [vp, i64, vp, i64, vp, vp, vp, i32, i64, i64, i32, i32, i32, dbl,
                                    vp, vp, vp, vp, vp, vp]
        _lib.fio_lookup.restype = None
        _lib.fio_compact.argtypes = [vp, vp, i64, vp]
        _lib.fio_compact.restype = i64
    return _lib


def set_threads(n: int) -> None:
    """Number of OpenMP threads the next calls use (1 = the paper's single-thread prototype, Sec. 5)."""
    rt = ctypes.CDLL("libgomp.so.1")
    rt.omp_set_num_threads(int(n))


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError("vectors must be float32 or uint16 (bf16 bit patterns)")


def sqdist(queries: np.ndarray, cache: np.ndarray) -> np.ndarray:
    """D[b][n] = sum_j (q_bj - c_nj)^2 in fp64."""
    q = np.ascontiguousarray(queries)
    x = np.ascontiguousarray(cache)
    assert q.dtype == x.dtype and q.shape[1] == x.shape[1]
    D = np.empty((q.shape[0], x.shape[0]), dtype=np.float64)
    _load().fio_sqdist(_ptr(q), _ptr(x), _dtype_code(x), q.shape[0], x.shape[0], x.shape[1], _ptr(D))
    return D


def select(D_row: np.ndarray, kk: int):
    """The kk smallest of one distance row under the order (D, n)."""
    D_row = np.ascontiguousarray(D_row, dtype=np.float64)
    kk = min(kk, D_row.shape[0])
    od = np.empty(max(kk, 1), dtype=np.float64)
    oi = np.empty(max(kk, 1), dtype=np.int64)
    if kk > 0:
        _load().fio_select(_ptr(D_row), D_row.shape[0], kk, _ptr(od), _ptr(oi))
    return od[:kk], oi[:kk]


def vote(nd: Sequence[float], nlabel: Sequence[int], nweight: Optional[Sequence[float]] = None, *,
         metric: int = METRIC_SQL2, rule: int = RULE_CONF_GT, tau: float = 0.0):
    """Label, confidence and hit from neighbour tuples given in ascending (distance, index) order."""
    nd = np.ascontiguousarray(nd, dtype=np.float64)
    nl = np.ascontiguousarray(nlabel, dtype=np.int32)
    nw = np.ones_like(nd) if nweight is None else np.ascontiguousarray(nweight, dtype=np.float64)
    label = ctypes.c_int32(0)
    conf = ctypes.c_double(0.0)
    hit = ctypes.c_uint8(0)
    _load().fio_vote(_ptr(nd), _ptr(nl), _ptr(nw), len(nd), metric, rule, float(tau),
                     ctypes.byref(label), ctypes.byref(conf), ctypes.byref(hit))
    return int(label.value), float(conf.value), bool(hit.value)


@dataclass
class LookupResult:
    label: np.ndarray      # [B] int32
    conf: np.ndarray       # [B] float64
    hit: np.ndarray        # [B] uint8
    nd: np.ndarray         # [B, k] float64 squared distances, ascending, +inf padded
    ni: np.ndarray         # [B, k] int64 cache indices, -1 padded
    next_d: np.ndarray     # [B] float64 squared distance of the (k+1)-th neighbour, +inf if none


def lookup(queries: np.ndarray, cache: np.ndarray, labels: np.ndarray, *, k: int, tau: float,
           rule: int = RULE_CONF_GT, metric: int = METRIC_SQL2, weights: Optional[np.ndarray] = None,
           row_idx: Optional[np.ndarray] = None) -> LookupResult:
    q = np.ascontiguousarray(queries)
    x = np.ascontiguousarray(cache)
    lab = np.ascontiguousarray(labels, dtype=np.int32)
    w = None if weights is None else np.ascontiguousarray(weights, dtype=np.float32)
    ridx = None if row_idx is None else np.ascontiguousarray(row_idx, dtype=np.int32)
    assert q.dtype == x.dtype and q.ndim == 2 and x.ndim == 2
    n, dim = x.shape
    assert q.shape[1] == dim and lab.shape[0] == n
    batch = q.shape[0] if ridx is None else ridx.shape[0]
    res = LookupResult(np.empty(batch, np.int32), np.empty(batch, np.float64), np.empty(batch, np.uint8),
                       np.empty((batch, k), np.float64), np.empty((batch, k), np.int64), np.empty(batch, np.float64))
    _load().fio_lookup(_ptr(q), q.shape[1], _ptr(ridx), batch, _ptr(x), _ptr(lab), _ptr(w), _dtype_code(x), n, dim,
                       int(k), int(metric), int(rule), float(tau), _ptr(res.label), _ptr(res.conf), _ptr(res.hit),
                       _ptr(res.nd), _ptr(res.ni), _ptr(res.next_d))
    return res


def compute_threshold(val_queries: np.ndarray, cache: np.ndarray, labels: np.ndarray, model_labels: np.ndarray, *,
                      k: int, metric: int = METRIC_SQL2, weights: Optional[np.ndarray] = None):
    """ComputeThresholds of Pseudocode 1 for one layer: walk the validation items in order and raise the
    threshold to the confidence of every look-up whose label is not the model's (Sec. 3.1 (ii)).  The paper
    leaves the starting value open; 0 is used.  Returns (threshold, number of wrong look-ups)."""
    r = lookup(val_queries, cache, labels, k=k, tau=0.0, metric=metric, weights=weights)
    threshold, wrong = 0.0, 0
    for item in range(r.label.shape[0]):
        if int(r.label[item]) != int(model_labels[item]):
            threshold = max(threshold, float(r.conf[item]))
            wrong += 1
    return threshold, wrong


@dataclass
class KMeansStep:
    assign: np.ndarray      # [n] int64 nearest-centre index of every point
    centres: np.ndarray     # [clusters, d] float64 means (old centre where a cluster is empty)
    counts: np.ndarray      # [clusters] int64
    majority: np.ndarray    # [clusters] int32, -1 for an empty cluster
    fraction: np.ndarray    # [clusters] float64 share of the majority label


def kmeans_step(points: np.ndarray, centres: np.ndarray, point_labels: np.ndarray, num_classes: int) -> KMeansStep:
    """One Lloyd iteration plus the tagging of Sec. 2.1 / Sec. 4: assign every point to its nearest centre (squared
    L2, ties to the smaller index), replace each centre by the mean of its points, and record per cluster the most
    frequent model-predicted label (smaller label on ties) with its share."""
    def stored_to_f64(a):
        return bf16_bits_to_f64(a) if a.dtype == np.uint16 else np.asarray(a, dtype=np.float64)
    clusters = centres.shape[0]
    r = lookup(points, centres, np.zeros(clusters, np.int32), k=1, tau=0.0)
    assign = r.ni[:, 0].copy()
    x = stored_to_f64(points)
    new = stored_to_f64(centres).copy()
    counts = np.zeros(clusters, np.int64)
    majority = np.full(clusters, -1, np.int32)
    fraction = np.zeros(clusters, np.float64)
    for c in range(clusters):
        members = np.nonzero(assign == c)[0]
        counts[c] = members.shape[0]
        if members.shape[0] == 0:
            continue
        new[c] = x[members].sum(axis=0) / members.shape[0]
        hist = np.bincount(point_labels[members], minlength=num_classes)
        majority[c] = int(np.argmax(hist))           # first maximum = smaller label on ties
        fraction[c] = hist[majority[c]] / members.shape[0]
    return KMeansStep(assign, new, counts, majority, fraction)


def merge_shards(shard_results: Sequence[LookupResult], shard_offsets: Sequence[int],
                 shard_labels: Sequence[np.ndarray], *, k: int, tau: float, rule: int = RULE_CONF_GT,
                 metric: int = METRIC_SQL2, shard_weights: Optional[Sequence[Optional[np.ndarray]]] = None) -> LookupResult:
    """Look-up against a cache whose rows are split into shards, from the shards' own look-up results: per query the
    shards' neighbour tuples are pooled under global row numbers, the k smallest under (D, n) kept, and the vote of
    Sec. 3 applied to them."""
    batch = shard_results[0].ni.shape[0]
    res = LookupResult(np.empty(batch, np.int32), np.empty(batch, np.float64), np.empty(batch, np.uint8),
                       np.full((batch, k), np.inf), np.full((batch, k), -1, np.int64), np.full(batch, np.inf))
    for b in range(batch):
        pool = []
        for s, r in enumerate(shard_results):
            for j in range(r.ni.shape[1]):
                li = int(r.ni[b, j])
                if li >= 0:
                    w = 1.0 if shard_weights is None or shard_weights[s] is None else float(shard_weights[s][li])
                    pool.append((float(r.nd[b, j]), li + int(shard_offsets[s]), int(shard_labels[s][li]), w))
        pool.sort(key=lambda t: (t[0], t[1]))
        top = pool[:k]
        lab, conf, hit = vote([t[0] for t in top], [t[2] for t in top], [t[3] for t in top], metric=metric, rule=rule,
                              tau=tau) if top else (-1, 0.0, False)
        res.label[b], res.conf[b], res.hit[b] = lab, conf, int(hit)
        for j, t in enumerate(top):
            res.nd[b, j], res.ni[b, j] = t[0], t[1]
        if len(pool) > k:
            res.next_d[b] = pool[k][0]
    return res


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) of float64 values, round to nearest, ties to even: the kept 16 bits are the top
    half of the float32 pattern, so the value is first rounded to the 8-bit significand directly from float64 (no
    double rounding through float32)."""
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros(x.shape, np.uint16)
    nz = np.isfinite(x) & (x != 0)
    m, e = np.frexp(np.abs(x[nz]))                       # |x| = m * 2**e, m in [0.5, 1)
    e_min = -126 + 1                                     # smallest normal exponent in frexp's convention
    shift = np.maximum(e, e_min)                         # below it the spacing stays that of the smallest normals
    q = np.abs(x[nz]) / np.ldexp(1.0, shift - 8)         # in units of the last kept bit: exact, a power-of-two scaling
    r = np.rint(q)                                       # numpy rounds halves to even
    val = (r * np.ldexp(1.0, shift - 8)).astype(np.float32)   # exactly representable in float32
    bits = (val.view(np.uint32) >> 16).astype(np.uint16)
    bits |= (np.signbit(x[nz]).astype(np.uint16) << 15)
    out[nz] = bits
    out[np.signbit(x) & (x == 0)] = 0x8000
    out[np.isposinf(x)] = 0x7F80
    out[np.isneginf(x)] = 0xFF80
    out[np.isnan(x)] = 0x7FC0
    return out


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def project(x: np.ndarray, weights: np.ndarray, bias: Optional[np.ndarray] = None):
    """Dimensionality reduction in front of the look-up (Sec. 3): y = max(0, W x + b) per row of x, in float64 on the
    stored values, then rounded once to bfloat16.  Returns (bf16 bit patterns [B, out], W x + b before the rectifier,
    sum_j |w_j x_j| + |b|: the magnitude a rounding-error bound scales with)."""
    xv = bf16_bits_to_f64(x) if x.dtype == np.uint16 else np.asarray(x, np.float64)
    wv = bf16_bits_to_f64(weights) if weights.dtype == np.uint16 else np.asarray(weights, np.float64)
    b = np.zeros(wv.shape[0]) if bias is None else np.asarray(bias, np.float64)
    pre = xv @ wv.T + b
    mag = np.abs(xv) @ np.abs(wv).T + np.abs(b)
    return round_to_bf16_bits(np.maximum(pre, 0.0)), pre, mag


def compact(active: np.ndarray, hit: np.ndarray) -> np.ndarray:
    """Ids of `active` whose look-up missed, order kept (Sec. 5, batch reconstruction)."""
    a = np.ascontiguousarray(active, dtype=np.int32)
    h = np.ascontiguousarray(hit, dtype=np.uint8)
    out = np.empty(max(1, a.shape[0]), dtype=np.int32)
    m = _load().fio_compact(_ptr(a), _ptr(h), a.shape[0], _ptr(out))
    return out[:m].copy()


@dataclass
class CascadeResult:
    final_label: np.ndarray    # [B0] int32, -1 = never frozen
    final_conf: np.ndarray     # [B0] float64
    exit_stage: np.ndarray     # [B0] int32, number of stages = never frozen
    active: List[np.ndarray]   # active[l] = request ids that reached stage l (ascending); one extra entry = survivors
    stage_results: List[LookupResult]


def cascade(stage_queries: Sequence[np.ndarray], stage_caches: Sequence[np.ndarray],
            stage_labels: Sequence[np.ndarray], taus: Sequence[float], *, k: int, rule: int = RULE_CONF_GT,
            metric: int = METRIC_SQL2, stage_weights: Optional[Sequence[Optional[np.ndarray]]] = None) -> CascadeResult:
    n_stage = len(stage_caches)
    b0 = stage_queries[0].shape[0]
    final_label = np.full(b0, -1, np.int32)
    final_conf = np.zeros(b0, np.float64)
    exit_stage = np.full(b0, n_stage, np.int32)
    active = [np.arange(b0, dtype=np.int32)]
    results = []
    for l in range(n_stage):
        ids = active[-1]
        w = None if stage_weights is None else stage_weights[l]
        r = lookup(stage_queries[l], stage_caches[l], stage_labels[l], k=k, tau=taus[l], rule=rule, metric=metric,
                   weights=w, row_idx=ids)
        frozen = r.hit.astype(bool)
        final_label[ids[frozen]] = r.label[frozen]
        final_conf[ids[frozen]] = r.conf[frozen]
        exit_stage[ids[frozen]] = l
        results.append(r)
        active.append(compact(ids, r.hit))
    return CascadeResult(final_label, final_conf, exit_stage, active, results)
