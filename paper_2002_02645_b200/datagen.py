"""Seeded synthetic activations for the per-layer cache look-up.

This module only draws inputs: labelled cache vectors, query vectors and the
class of every request.  It holds none of the look-up arithmetic (no distance,
no vote, no threshold rule), so the CUDA path and the CPU oracle can both be
fed from it without sharing any of the method.

Random numbers come from numpy's Philox counter-based generator, keyed by
(seed, stream id, chunk index).  Rows are produced in fixed-size chunks, each
chunk from its own key, so the values do not depend on the number of worker
threads that fill them.

Storage types
-------------
"f32"  : numpy float32
"bf16" : numpy uint16 holding the upper half of the float32 pattern after an
         explicit round-to-nearest-even; both sides read exactly these bits.

The shapes follow the workloads the paper describes: ResNet-18 block outputs
of 64x32x32 ... 512x4x4 values per image (Sec. 2.1 and Table 1 give 8 blocks
and the cache footprint they add up to), pooled ResNet-50 stage outputs, and
tens of thousands of cached entries per layer (Sec. 4).  CIFAR / ImageNet
activations themselves are not available; labelled mixtures stand in for them.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

# stream ids: one namespace per kind of draw so that no two draws share a key
_S_MEANS, _S_CACHE_LABELS, _S_CACHE_NOISE = 1, 2, 3
_S_QUERY_LABELS, _S_QUERY_NOISE, _S_COPIES, _S_SHUFFLE = 4, 5, 6, 7
_S_PROJ_W, _S_PROJ_B = 8, 9

_CHUNK_ELEMS = 1 << 22


def _rng(seed: int, stream: int, stage: int = 0, chunk: int = 0) -> np.random.Generator:
    key = (np.uint64(seed) << np.uint64(32)) | np.uint64(stream & 0xFFFF) << np.uint64(16) | np.uint64(stage & 0xFFFF)
    return np.random.Generator(np.random.Philox(key=[int(key), int(chunk)]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def stored_to_f64(x: np.ndarray) -> np.ndarray:
    """Exact fp64 value of stored vectors (float32 array or bf16 bit patterns)."""
    if x.dtype == np.uint16:
        return bf16_bits_to_f32(x).astype(np.float64)
    return x.astype(np.float64)


def _workers() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def class_probs(num_classes: int, zipf: Optional[float]) -> np.ndarray:
    """Uniform class frequencies, or p_c proportional to (c+1)^-zipf."""
    if zipf is None:
        return np.full(num_classes, 1.0 / num_classes)
    p = (np.arange(num_classes, dtype=np.float64) + 1.0) ** (-float(zipf))
    return p / p.sum()


def draw_labels(n: int, probs: np.ndarray, seed: int, stream: int, stage: int = 0) -> np.ndarray:
    g = _rng(seed, stream, stage)
    cdf = np.cumsum(probs)
    cdf[-1] = 1.0
    return np.searchsorted(cdf, g.random(n), side="right").astype(np.int32)


def class_means(num_classes: int, dim: int, seed: int, stage: int) -> np.ndarray:
    """One N(0,1)^dim vector per (stage, class), float32."""
    g = _rng(seed, _S_MEANS, stage)
    return g.standard_normal((num_classes, dim), dtype=np.float32)


def _fill_rows(out: np.ndarray, labels: np.ndarray, means: np.ndarray, *, kind: str, scale: float,
               seed: int, stream: int, stage: int, dtype: str) -> None:
    """Fill `out` row by row.

    kind == "relu_mixture": x = max(0, mean_c + scale * eps)
    kind == "halfnormal"  : x = | eps + scale * mean_c |
    """
    n, dim = out.shape
    rows_per_chunk = max(1, _CHUNK_ELEMS // dim)
    chunks = [(c, lo, min(n, lo + rows_per_chunk)) for c, lo in enumerate(range(0, n, rows_per_chunk))]

    def work(item):
        c, lo, hi = item
        g = _rng(seed, stream, stage, c)
        eps = g.standard_normal((hi - lo, dim), dtype=np.float32)
        mu = means[labels[lo:hi]]
        if kind == "relu_mixture":
            eps *= np.float32(scale)
            eps += mu
            np.maximum(eps, np.float32(0.0), out=eps)
        elif kind == "halfnormal":
            eps += np.float32(scale) * mu
            np.abs(eps, out=eps)
        else:  # pragma: no cover
            raise ValueError(kind)
        out[lo:hi] = f32_to_bf16_bits(eps) if dtype == "bf16" else eps

    if len(chunks) == 1:
        work(chunks[0])
    else:
        with ThreadPoolExecutor(_workers()) as ex:
            list(ex.map(work, chunks))


def projection_weights(in_dim: int, out_dim: int, seed: int, stage: int = 0):
    """Random stand-in for a layer's trained dimensionality-reduction weights (the trained ones are not available):
    W [out_dim, in_dim] ~ N(0, 1/in_dim) as bf16 bit patterns, bias [out_dim] ~ 0.1 N(0, 1) as float32."""
    w = np.empty((out_dim, in_dim), dtype=np.uint16)
    rows_per_chunk = max(1, _CHUNK_ELEMS // in_dim)
    scale = np.float32(1.0 / np.sqrt(in_dim))
    for c, lo in enumerate(range(0, out_dim, rows_per_chunk)):
        hi = min(out_dim, lo + rows_per_chunk)
        w[lo:hi] = f32_to_bf16_bits(_rng(seed, _S_PROJ_W, stage, c).standard_normal((hi - lo, in_dim), dtype=np.float32) * scale)
    bias = (_rng(seed, _S_PROJ_B, stage).standard_normal(out_dim, dtype=np.float32) * np.float32(0.1)).astype(np.float32)
    return w, bias


def _alloc(n: int, dim: int, dtype: str) -> np.ndarray:
    return np.empty((n, dim), dtype=np.uint16 if dtype == "bf16" else np.float32)


@dataclass
class StageData:
    """One layer: its cache and the activations of every request at that layer."""
    dim: int
    dtype: str                 # "f32" | "bf16"
    cache_vecs: np.ndarray     # [N, dim]  float32 or uint16 (bf16 bits)
    cache_labels: np.ndarray   # [N] int32
    queries: np.ndarray        # [B0, dim]
    calib: Optional[np.ndarray] = None   # [Bc, dim] separate draws for setting thresholds


@dataclass
class Workload:
    name: str
    num_classes: int
    k: int
    stages: List[StageData]
    query_classes: np.ndarray            # [B0] class each request was drawn from
    calib_classes: Optional[np.ndarray] = None
    meta: Dict[str, object] = field(default_factory=dict)


def make_stage(*, n_cache: int, n_query: int, n_calib: int, dim: int, num_classes: int, dtype: str, kind: str,
               scale: float, seed: int, stage: int, probs: np.ndarray,
               query_classes: Optional[np.ndarray] = None, calib_classes: Optional[np.ndarray] = None,
               query_seed: Optional[int] = None):
    """`query_seed` (default: `seed`) draws another batch of requests against the same cache."""
    qseed = seed if query_seed is None else query_seed
    means = class_means(num_classes, dim, seed, stage)
    cache_labels = draw_labels(n_cache, probs, seed, _S_CACHE_LABELS, stage)
    cache = _alloc(n_cache, dim, dtype)
    _fill_rows(cache, cache_labels, means, kind=kind, scale=scale, seed=seed, stream=_S_CACHE_NOISE,
               stage=stage, dtype=dtype)
    if query_classes is None:
        query_classes = draw_labels(n_query, probs, qseed, _S_QUERY_LABELS, 0)
    queries = _alloc(n_query, dim, dtype)
    _fill_rows(queries, query_classes, means, kind=kind, scale=scale, seed=qseed, stream=_S_QUERY_NOISE,
               stage=stage, dtype=dtype)
    calib = None
    if n_calib > 0:
        if calib_classes is None:
            calib_classes = draw_labels(n_calib, probs, seed + 1, _S_QUERY_LABELS, 0)
        calib = _alloc(n_calib, dim, dtype)
        _fill_rows(calib, calib_classes, means, kind=kind, scale=scale, seed=seed + 1, stream=_S_QUERY_NOISE,
                   stage=stage, dtype=dtype)
    return StageData(dim, dtype, cache, cache_labels, queries, calib), query_classes, calib_classes


def single_layer(*, name: str, n_cache: int, n_query: int, dim: int, num_classes: int, dtype: str, sigma: float,
                 k: int, seed: int = 0, n_copies: int = 0, n_calib: int = 0, zipf: Optional[float] = None,
                 query_seed: Optional[int] = None) -> Workload:
    """One cache of ReLU'd Gaussian-mixture vectors; optional exact copies of cache rows among the queries."""
    probs = class_probs(num_classes, zipf)
    st, qc, cc = make_stage(n_cache=n_cache, n_query=n_query, n_calib=n_calib, dim=dim, num_classes=num_classes,
                            dtype=dtype, kind="relu_mixture", scale=sigma, seed=seed, stage=0, probs=probs,
                            query_seed=query_seed)
    meta: Dict[str, object] = {}
    if n_copies > 0:
        g = _rng(seed, _S_COPIES)
        src = g.integers(0, n_cache, size=n_copies)
        q = np.concatenate([st.queries, st.cache_vecs[src]], axis=0)
        qc = np.concatenate([qc, st.cache_labels[src]])
        copy_of = np.concatenate([np.full(n_query, -1, dtype=np.int64), src.astype(np.int64)])
        perm = _rng(seed, _S_SHUFFLE).permutation(q.shape[0])
        st.queries = np.ascontiguousarray(q[perm])
        qc = qc[perm]
        meta["copy_of"] = copy_of[perm]
    return Workload(name, num_classes, k, [st], qc, cc, meta)


def cascade(*, name: str, dims: List[int], scales: List[float], kind: str, n_cache: int, n_query: int, n_calib: int,
            num_classes: int, dtype: str, k: int, seed: int = 0, zipf: Optional[float] = None,
            query_seed: Optional[int] = None) -> Workload:
    """One cache per stage; the class of request r is the same at every stage."""
    probs = class_probs(num_classes, zipf)
    stages: List[StageData] = []
    qc = cc = None
    for s, (dim, scale) in enumerate(zip(dims, scales)):
        st, qc, cc = make_stage(n_cache=n_cache, n_query=n_query, n_calib=n_calib, dim=dim, num_classes=num_classes,
                                dtype=dtype, kind=kind, scale=scale, seed=seed, stage=s, probs=probs,
                                query_classes=qc, calib_classes=cc, query_seed=query_seed)
        stages.append(st)
    return Workload(name, num_classes, k, stages, qc, cc, {"scales": list(scales)})


# ----------------------------------------------------------------------------------------------
# The five named workloads.  `shrink` divides entry and batch counts (and, for the two deep
# cascades, the vector length) so that the same recipe also gives cases a CPU can finish in seconds.
# ----------------------------------------------------------------------------------------------

def config1(seed: int = 0) -> Workload:
    """1,000 fp32 vectors of 512 values, 10 classes, sigma 0.5, ReLU; 256 fresh queries + 26 exact copies; k = 1."""
    w = single_layer(name="cfg1_single_layer_f32", n_cache=1000, n_query=256, dim=512, num_classes=10, dtype="f32",
                     sigma=0.5, k=1, seed=seed, n_copies=26)
    w.meta["rule"] = "dist_le"
    return w


def config2(seed: int = 0, shrink: int = 1, n_calib: int = 512, query_seed: Optional[int] = None,
            stages: int = 4) -> Workload:
    """Four-stage ResNet-18/CIFAR-10-shaped cascade, bf16, half-normal values with growing class shifts; k = 5."""
    dims = [65536 // shrink, 32768 // shrink, 16384 // shrink, 8192 // shrink][:stages]
    w = cascade(name="cfg2_resnet18_cascade" + ("" if shrink == 1 else f"_shrink{shrink}"), dims=dims,
                scales=[0.2, 0.4, 0.8, 1.6][:stages], kind="halfnormal", n_cache=10000 // shrink, n_query=1024 // shrink,
                n_calib=n_calib // shrink, num_classes=10, dtype="bf16", k=5, seed=seed, query_seed=query_seed)
    w.meta.update(rule="conf_gt", percentiles=[80.0, 60.0, 40.0, 20.0][:stages])
    return w


def config3(seed: int = 0, shrink: int = 1, n_calib: int = 512, query_seed: Optional[int] = None,
            n_cache: Optional[int] = None) -> Workload:
    """One layer, 200,000 bf16 entries of 8192 values, sigma 0.7, ReLU; batch 8,192; k = 10.  `n_cache` keeps the batch
    and takes only the first entries' worth of the cache (profiler captures on a smaller footprint)."""
    w = single_layer(name="cfg3_large_cache" + ("" if shrink == 1 else f"_shrink{shrink}"),
                     n_cache=(200000 // shrink) if n_cache is None else n_cache,
                     n_query=8192 // shrink, dim=8192, num_classes=10, dtype="bf16", sigma=0.7, k=10, seed=seed,
                     n_calib=max(1, n_calib // shrink), query_seed=query_seed)
    w.meta.update(rule="conf_gt", percentiles=[50.0])
    return w


def config4(seed: int = 0, shrink: int = 1, n_calib: int = 512, query_seed: Optional[int] = None,
            stages: int = 4, first_stage: int = 0) -> Workload:
    """Four-stage ImageNet-shaped cascade: 100,000 entries per stage, 1,000 Zipf(1.1) classes, sigma 0.6; k = 5.
    `first_stage` / `stages` cut out a run of stages (one stage alone: a profiler capture of its kernel)."""
    w = cascade(name="cfg4_imagenet_cascade" + ("" if shrink == 1 else f"_shrink{shrink}"),
                dims=[256, 512, 1024, 2048][first_stage:first_stage + stages], scales=[0.6] * stages, kind="relu_mixture", n_cache=100000 // shrink,
                n_query=4096 // shrink, n_calib=max(1, n_calib // shrink), num_classes=1000, dtype="bf16", k=5,
                seed=seed, zipf=1.1, query_seed=query_seed)
    w.meta.update(rule="conf_gt", percentiles=[80.0, 60.0, 40.0, 20.0][first_stage:first_stage + stages])
    return w


def config5(seed: int = 0, shrink: int = 1, batch: int = 16, query_seed: Optional[int] = None) -> Workload:
    """Latency regime: 50,000 bf16 entries of 16384 values, sigma 0.5, ReLU; batches of 1, 4, 16; k = 1."""
    w = single_layer(name="cfg5_latency" + ("" if shrink == 1 else f"_shrink{shrink}"), n_cache=50000 // shrink,
                     n_query=batch, dim=16384, num_classes=10, dtype="bf16", sigma=0.5, k=1, seed=seed,
                     query_seed=query_seed)
    w.meta["rule"] = "dist_le"
    return w
