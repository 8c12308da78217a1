"""Thin ctypes binding of the C ABI in include/fi.h.

Only argument marshalling happens here: torch tensors provide device memory and the current CUDA stream;
every step of a look-up runs in the library's kernels.  Loading fails loudly when the library is missing:
there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

from . import build as _build

FI_OK = 0
FI_ERR_INVALID_ARG, FI_ERR_CAPACITY, FI_ERR_OOM, FI_ERR_CUDA, FI_ERR_UNSUPPORTED, FI_ERR_TIMEOUT = 1, 2, 3, 4, 5, 6
FI_F32, FI_BF16 = 0, 1
FI_HIT_CONF_GT, FI_HIT_DIST_LE = 0, 1
FI_METRIC_SQL2, FI_METRIC_L2 = 0, 1
FI_PATH_AUTO, FI_PATH_STREAM, FI_PATH_GEMM = 0, 1, 2

EXPORTS = ["fi_cache_create", "fi_cache_destroy", "fi_cache_insert", "fi_cache_set_threshold", "fi_cache_set_path",
           "fi_cache_size", "fi_cache_lookup_batch", "fi_cascade_init", "fi_cascade_step", "fi_cache_lookup_batch_host",
           "fi_cascade_run_host", "fi_cache_poll_status", "fi_cache_set_profiling",
           "fi_cache_read_profile", "fi_lookup_noalloc", "fi_cache_compute_threshold", "fi_cache_clear", "fi_kmeans_step", "fi_cache_selftest_wait", "fi_cache_neighbor_tuples", "fi_merge_shard_lookups",
           "fi_projection_create", "fi_projection_destroy", "fi_projection_set_weights", "fi_projection_apply", "fi_projection_poll_status", "fi_projection_set_profiling",
           "fi_projection_read_profile",
           "fi_cascade_step_projected", "fi_cache_set_repair", "fi_cache_read_certificate",
           "fi_cache_read_slot_certificates", "fi_cache_lookup_view", "fi_cache_set_sm_limit", "fi_gemm_plan_describe", "fi_launch_count", "fi_last_error", "fi_status_string"]


class fi_cache_config_t(ctypes.Structure):
    _fields_ = [("dim", ctypes.c_int32), ("dtype", ctypes.c_int32), ("capacity", ctypes.c_int64),
                ("num_classes", ctypes.c_int32), ("k", ctypes.c_int32), ("rule", ctypes.c_int32),
                ("metric", ctypes.c_int32), ("threshold", ctypes.c_float), ("device", ctypes.c_int32),
                ("max_batch", ctypes.c_int32), ("path", ctypes.c_int32)]


class fi_lookup_out_t(ctypes.Structure):
    _fields_ = [("label", ctypes.c_void_p), ("conf", ctypes.c_void_p), ("hit", ctypes.c_void_p),
                ("topk_dist", ctypes.c_void_p), ("topk_idx", ctypes.c_void_p)]


class fi_cascade_state_t(ctypes.Structure):
    _fields_ = [("active_idx", ctypes.c_void_p), ("active_count", ctypes.c_void_p), ("miss_idx", ctypes.c_void_p),
                ("miss_count", ctypes.c_void_p), ("final_label", ctypes.c_void_p), ("exit_stage", ctypes.c_void_p),
                ("final_conf", ctypes.c_void_p), ("stage", ctypes.c_int32), ("batch0", ctypes.c_int32)]


class FiError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{status_string(status)}: {message}")
        self.status = status


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen libficache.so (built in-tree by `build.build_library`) and declare the prototypes."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _build.LIB
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} is missing: build it with paper_2002_02645_b200.build.build_library()")
    lib = ctypes.CDLL(path)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.fi_cache_create.argtypes = [ctypes.POINTER(fi_cache_config_t), ctypes.POINTER(vp)]
    lib.fi_cache_destroy.argtypes = [vp]
    lib.fi_cache_insert.argtypes = [vp, vp, vp, vp, i64, vp]
    lib.fi_cache_set_threshold.argtypes = [vp, ctypes.c_float]
    lib.fi_cache_set_path.argtypes = [vp, i32]
    lib.fi_cache_size.argtypes = [vp]
    lib.fi_cache_size.restype = i64
    lib.fi_cache_lookup_batch.argtypes = [vp, vp, i64, vp, i32, vp, ctypes.POINTER(fi_lookup_out_t), vp]
    lib.fi_cascade_init.argtypes = [ctypes.POINTER(fi_cascade_state_t), i32, i32, vp]
    lib.fi_cascade_step.argtypes = [vp, vp, i64, ctypes.POINTER(fi_cascade_state_t), vp]
    lib.fi_cache_lookup_batch_host.argtypes = [vp, vp, i32, ctypes.POINTER(fi_lookup_out_t), vp]
    lib.fi_cascade_run_host.argtypes = [ctypes.POINTER(vp), i32, ctypes.POINTER(vp), i32, vp, vp, vp, vp, vp]
    lib.fi_cache_poll_status.argtypes = [vp]
    lib.fi_cache_clear.argtypes = [vp]
    lib.fi_cache_neighbor_tuples.argtypes = [vp, vp, i64, i32, vp, vp, vp, vp]
    lib.fi_merge_shard_lookups.argtypes = [i32, i32, i32, vp, vp, vp, vp, i32, i32, ctypes.c_float,
                                           ctypes.POINTER(fi_lookup_out_t), vp]
    lib.fi_projection_create.argtypes = [i32, i32, i32, i32, ctypes.POINTER(vp)]
    lib.fi_projection_destroy.argtypes = [vp]
    lib.fi_projection_set_weights.argtypes = [vp, vp, vp, vp]
    lib.fi_projection_poll_status.argtypes = [vp]
    lib.fi_projection_set_profiling.argtypes = [vp, i32]
    lib.fi_projection_read_profile.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
    lib.fi_projection_apply.argtypes = [vp, vp, i64, vp, i32, vp, vp, i64, vp]
    lib.fi_cascade_step_projected.argtypes = [vp, vp, vp, i64, ctypes.POINTER(fi_cascade_state_t), vp]
    lib.fi_cache_selftest_wait.argtypes = [vp, i64, vp]
    lib.fi_kmeans_step.argtypes = [vp, vp, i64, vp, i64, vp, vp, vp, vp, vp, vp]
    lib.fi_cache_compute_threshold.argtypes = [vp, vp, i64, vp, i64, ctypes.POINTER(ctypes.c_float),
                                               ctypes.POINTER(i64), vp]
    lib.fi_lookup_noalloc.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, i32, ctypes.c_float, vp, i64, i32,
                                      ctypes.POINTER(fi_lookup_out_t), vp]
    lib.fi_cache_lookup_view.argtypes = [vp]
    lib.fi_cache_lookup_view.restype = i64
    lib.fi_cache_set_sm_limit.argtypes = [vp, i32]
    lib.fi_cache_set_repair.argtypes = [vp, i32]
    lib.fi_cache_read_certificate.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(ctypes.c_float)]
    lib.fi_cache_read_slot_certificates.argtypes = [vp, vp, i32]
    lib.fi_cache_set_profiling.argtypes = [vp, i32]
    lib.fi_cache_read_profile.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
    lib.fi_gemm_plan_describe.argtypes = [i32, i64, i32, i32, i32, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                          ctypes.POINTER(i32)]
    lib.fi_gemm_plan_describe.restype = i32
    lib.fi_launch_count.argtypes = []
    lib.fi_launch_count.restype = i64
    lib.fi_last_error.argtypes = []
    lib.fi_last_error.restype = ctypes.c_char_p
    lib.fi_status_string.argtypes = [i32]
    lib.fi_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is ctypes.c_int:   # default: the fi_status_t functions
            fn.restype = i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().fi_status_string(int(status)).decode()


def _check(status: int) -> None:
    if status != FI_OK:
        raise FiError(status, load_library().fi_last_error().decode())


PLAN_FIELDS = ("count", "m_tiles", "mg", "groups", "parts", "range16", "list_len", "tile_m", "lists", "mode", "n_tiles",
               "tail_tiles", "tail_slices", "pieces", "half", "span_full", "span_half")


def gemm_plan_describe(count: int, n_entries: int, num_ctas: int, k: int, dim: int, max_batch: int, cta: int = -1):
    """Host only: the work split of the distance GEMM as a dict, plus (spans mode, cta >= 0) that CTA's pieces as
    tuples (query tile, cache-row tile, first k-block, end k-block, 128-row MMAs, slot)."""
    plan = (ctypes.c_int32 * 17)()
    items = (ctypes.c_int32 * 18)()
    n = ctypes.c_int32(0)
    _check(load_library().fi_gemm_plan_describe(count, n_entries, num_ctas, k, dim, max_batch, cta, plan, items,
                                                ctypes.byref(n)))
    return dict(zip(PLAN_FIELDS, plan)), [tuple(items[6 * i:6 * i + 6]) for i in range(n.value)]


def launch_count() -> int:
    return int(load_library().fi_launch_count())


def _stream_ptr(device: torch.device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _dp(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


_TORCH_DTYPE = {FI_F32: torch.float32, FI_BF16: torch.bfloat16}


class LookupOut:
    """Device arrays a look-up writes (torch owns the memory)."""

    def __init__(self, batch: int, k: int, device, with_topk: bool = True):
        self.label = torch.empty(batch, dtype=torch.int32, device=device)
        self.conf = torch.empty(batch, dtype=torch.float32, device=device)
        self.hit = torch.empty(batch, dtype=torch.uint8, device=device)
        self.topk_dist = torch.empty(batch, k, dtype=torch.float32, device=device) if with_topk else None
        self.topk_idx = torch.empty(batch, k, dtype=torch.int32, device=device) if with_topk else None

    def as_struct(self) -> fi_lookup_out_t:
        return fi_lookup_out_t(_dp(self.label), _dp(self.conf), _dp(self.hit), _dp(self.topk_dist), _dp(self.topk_idx))


class FreezeCache:
    """CACHE[layer] and THRESHOLDS[layer] of one layer, resident on one GPU."""

    def __init__(self, *, dim: int, capacity: int, num_classes: int, k: int, dtype: int = FI_BF16,
                 rule: int = FI_HIT_CONF_GT, metric: int = FI_METRIC_SQL2, threshold: float = 0.0, device: int = 0,
                 max_batch: int = 1024, path: int = FI_PATH_AUTO):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        self.cfg = fi_cache_config_t(dim, dtype, capacity, num_classes, k, rule, metric, threshold, device, max_batch, path)
        self.device = torch.device("cuda", device)
        _check(self._lib.fi_cache_create(ctypes.byref(self.cfg), ctypes.byref(self._h)))

    # -- fi_cache_destroy
    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.fi_cache_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self) -> ctypes.c_void_p:
        return self._h

    @property
    def k(self) -> int:
        return self.cfg.k

    @property
    def dim(self) -> int:
        return self.cfg.dim

    def _check_vecs(self, t: torch.Tensor) -> None:
        if t.device != self.device or t.dtype != _TORCH_DTYPE[self.cfg.dtype] or t.dim() != 2 or t.shape[1] != self.cfg.dim \
                or t.stride(1) != 1:
            raise ValueError("vectors must be a 2-D tensor of the cache's dtype, dim and device with unit inner stride")

    # -- fi_cache_insert
    def insert(self, vecs: torch.Tensor, labels: torch.Tensor, weights: Optional[torch.Tensor] = None) -> None:
        self._check_vecs(vecs)
        if not vecs.is_contiguous():
            raise ValueError("inserted rows must be contiguous")
        if labels.dtype != torch.int32 or labels.device != self.device or labels.numel() != vecs.shape[0]:
            raise ValueError("labels must be int32 on the cache's device, one per row")
        if weights is not None and (weights.dtype != torch.float32 or weights.device != self.device
                                    or weights.numel() != vecs.shape[0]):
            raise ValueError("weights must be float32 on the cache's device, one per row")
        _check(self._lib.fi_cache_insert(self._h, _dp(vecs), _dp(labels), _dp(weights), vecs.shape[0],
                                         _stream_ptr(self.device)))

    # -- fi_cache_set_threshold / fi_cache_set_path / fi_cache_size / fi_cache_poll_status
    def set_threshold(self, tau: float) -> None:
        _check(self._lib.fi_cache_set_threshold(self._h, float(tau)))
        self.cfg.threshold = float(tau)

    def set_path(self, path: int) -> None:
        _check(self._lib.fi_cache_set_path(self._h, int(path)))

    def size(self) -> int:
        return int(self._lib.fi_cache_size(self._h))

    def poll_status(self) -> None:
        _check(self._lib.fi_cache_poll_status(self._h))

    # -- fi_cache_lookup_view / fi_cache_set_sm_limit
    def lookup_view(self) -> int:
        """Entries the most recent look-up covered (inserts still in flight on another stream are not among them)."""
        return int(self._lib.fi_cache_lookup_view(self._h))

    def set_sm_limit(self, sms: int) -> None:
        _check(self._lib.fi_cache_set_sm_limit(self._h, int(sms)))

    # -- fi_cache_set_repair / fi_cache_read_certificate / fi_cache_read_slot_certificates
    def set_repair(self, enable: bool) -> None:
        _check(self._lib.fi_cache_set_repair(self._h, 1 if enable else 0))

    def read_certificate(self):
        """(requests without a certificate since the last read, of those not repaired, largest observed score error)."""
        unc, unrep, err = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_float(0.0)
        _check(self._lib.fi_cache_read_certificate(self._h, ctypes.byref(unc), ctypes.byref(unrep), ctypes.byref(err)))
        return int(unc.value), int(unrep.value), float(err.value)

    def slot_certificates(self, n: int) -> torch.Tensor:
        """Flags of the most recent look-up, slots 0..n-1 (host uint8 tensor, 1 = certified or repaired)."""
        flags = torch.zeros(max(n, 1), dtype=torch.uint8)
        _check(self._lib.fi_cache_read_slot_certificates(self._h, flags.data_ptr(), int(n)))
        return flags[:n]

    # -- fi_cache_neighbor_tuples
    def neighbor_tuples(self, topk_idx: torch.Tensor, index_offset: int):
        """(global index, label, weight) of the neighbours a look-up on this shard returned."""
        n = topk_idx.numel()
        gi = torch.empty_like(topk_idx)
        lab = torch.empty_like(topk_idx)
        wgt = torch.empty(topk_idx.shape, dtype=torch.float32, device=self.device)
        _check(self._lib.fi_cache_neighbor_tuples(self._h, _dp(topk_idx), n, int(index_offset), _dp(gi), _dp(lab), _dp(wgt),
                                                  _stream_ptr(self.device)))
        return gi, lab, wgt

    # -- fi_cache_selftest_wait
    def selftest_wait(self, limit_cycles: int = 2_000_000) -> None:
        """Enqueue the bounded-wait self-test; the next poll_status() raises FI_ERR_TIMEOUT."""
        _check(self._lib.fi_cache_selftest_wait(self._h, int(limit_cycles), _stream_ptr(self.device)))

    # -- fi_cache_clear
    def clear(self) -> None:
        _check(self._lib.fi_cache_clear(self._h))

    # -- fi_kmeans_step
    def kmeans_step(self, points: torch.Tensor, point_labels: torch.Tensor):
        """One Lloyd iteration with this cache's entries as the current centres (k must be 1).
        Returns (assignment [n], new centres [size, dim], counts [size], majority label [size], fraction [size])."""
        self._check_vecs(points)
        n, size = points.shape[0], self.size()
        assign = torch.empty(max(n, 1), dtype=torch.int32, device=self.device)
        centres = torch.empty(size, self.cfg.dim, dtype=_TORCH_DTYPE[self.cfg.dtype], device=self.device)
        counts = torch.empty(size, dtype=torch.int32, device=self.device)
        majority = torch.empty(size, dtype=torch.int32, device=self.device)
        fraction = torch.empty(size, dtype=torch.float32, device=self.device)
        _check(self._lib.fi_kmeans_step(self._h, _dp(points), points.stride(0), _dp(point_labels), n, _dp(assign),
                                        _dp(centres), _dp(counts), _dp(majority), _dp(fraction),
                                        _stream_ptr(self.device)))
        return assign[:n], centres, counts, majority, fraction

    # -- fi_cache_compute_threshold
    def compute_threshold(self, val_acts: torch.Tensor, model_labels: torch.Tensor):
        """ComputeThresholds for this layer: (threshold now set on the cache, number of wrong look-ups)."""
        self._check_vecs(val_acts)
        if model_labels.dtype != torch.int32 or model_labels.device != self.device \
                or model_labels.numel() != val_acts.shape[0]:
            raise ValueError("model_labels must be int32 on the cache's device, one per validation item")
        tau, wrong = ctypes.c_float(0.0), ctypes.c_int64(0)
        _check(self._lib.fi_cache_compute_threshold(self._h, _dp(val_acts), val_acts.stride(0), _dp(model_labels),
                                                    val_acts.shape[0], ctypes.byref(tau), ctypes.byref(wrong),
                                                    _stream_ptr(self.device)))
        return float(tau.value), int(wrong.value)

    # -- fi_cache_set_profiling / fi_cache_read_profile
    def set_profiling(self, enable: bool) -> None:
        _check(self._lib.fi_cache_set_profiling(self._h, 1 if enable else 0))

    def read_profile(self):
        """(summed distance-kernel milliseconds, launches covered) since the last read."""
        ms, n = ctypes.c_float(0.0), ctypes.c_int32(0)
        _check(self._lib.fi_cache_read_profile(self._h, ctypes.byref(ms), ctypes.byref(n)))
        return float(ms.value), int(n.value)

    # -- fi_cache_lookup_batch
    def lookup_batch(self, queries: torch.Tensor, *, row_idx: Optional[torch.Tensor] = None,
                     batch_max: Optional[int] = None, batch_count: Optional[torch.Tensor] = None,
                     out: Optional[LookupOut] = None, with_topk: bool = True) -> LookupOut:
        self._check_vecs(queries)
        if batch_max is None:
            batch_max = int(row_idx.numel()) if row_idx is not None else int(queries.shape[0])
        if out is None:
            out = LookupOut(batch_max, self.cfg.k, self.device, with_topk)
        st = out.as_struct()
        _check(self._lib.fi_cache_lookup_batch(self._h, _dp(queries), queries.stride(0), _dp(row_idx), batch_max,
                                               _dp(batch_count), ctypes.byref(st), _stream_ptr(self.device)))
        return out

    # -- fi_cache_lookup_batch_host
    def lookup_batch_host(self, queries_host: torch.Tensor, out_host: LookupOut) -> LookupOut:
        """queries_host and the arrays of out_host live in (pinned) host memory."""
        if queries_host.is_cuda or not queries_host.is_contiguous() or queries_host.shape[1] != self.cfg.dim:
            raise ValueError("queries_host must be a contiguous host tensor [batch, dim]")
        st = out_host.as_struct()
        _check(self._lib.fi_cache_lookup_batch_host(self._h, _dp(queries_host), queries_host.shape[0], ctypes.byref(st),
                                                    _stream_ptr(self.device)))
        return out_host


def lookup_noalloc(cache_vecs: torch.Tensor, labels: torch.Tensor, weights: torch.Tensor, queries: torch.Tensor, *,
                   k: int, rule: int = FI_HIT_CONF_GT, metric: int = FI_METRIC_SQL2, threshold: float = 0.0,
                   out: Optional[LookupOut] = None) -> LookupOut:
    """fi_lookup_noalloc: the streaming look-up on plain device arrays, scratch inside the library image.
    For callers that cannot allocate device memory; `weights` is required (ones for a plain k-NN cache).
    At most 256 requests per call; calls on one device must not overlap on the GPU."""
    dtype = FI_BF16 if cache_vecs.dtype == torch.bfloat16 else FI_F32
    if queries.dtype != cache_vecs.dtype or queries.dim() != 2 or cache_vecs.dim() != 2 or queries.stride(1) != 1 \
            or not cache_vecs.is_contiguous():
        raise ValueError("cache_vecs and queries must be 2-D tensors of one dtype; cache rows contiguous")
    dev = cache_vecs.device
    if out is None:
        out = LookupOut(queries.shape[0], k, dev)
    st = out.as_struct()
    with torch.cuda.device(dev):
        _check(load_library().fi_lookup_noalloc(_dp(cache_vecs), _dp(labels), _dp(weights), cache_vecs.shape[0],
                                                cache_vecs.shape[1], dtype, k, rule, metric, float(threshold),
                                                _dp(queries), queries.stride(0), queries.shape[0], ctypes.byref(st),
                                                _stream_ptr(dev)))
    return out


class Projection:
    """The dimensionality reduction in front of the look-up (Sec. 3): y = max(0, W x + b) in bf16."""

    def __init__(self, *, in_dim: int, out_dim: int = 1024, device: int = 0, max_batch: int = 1024):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        self.in_dim, self.out_dim, self.max_batch = in_dim, out_dim, max_batch
        self.device = torch.device("cuda", device)
        _check(self._lib.fi_projection_create(in_dim, out_dim, device, max_batch, ctypes.byref(self._h)))

    # -- fi_projection_destroy
    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.fi_projection_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self) -> ctypes.c_void_p:
        return self._h

    # -- fi_projection_set_weights
    def set_weights(self, weights: torch.Tensor, bias: Optional[torch.Tensor] = None) -> None:
        if weights.dtype != torch.bfloat16 or tuple(weights.shape) != (self.out_dim, self.in_dim) \
                or not weights.is_contiguous() or weights.device != self.device:
            raise ValueError("weights must be a contiguous bf16 [out_dim, in_dim] tensor on the projection's device")
        if bias is not None and (bias.dtype != torch.float32 or bias.numel() != self.out_dim or bias.device != self.device):
            raise ValueError("bias must be float32 [out_dim] on the projection's device")
        _check(self._lib.fi_projection_set_weights(self._h, _dp(weights), _dp(bias), _stream_ptr(self.device)))

    # -- fi_projection_poll_status
    def poll_status(self) -> None:
        _check(self._lib.fi_projection_poll_status(self._h))

    # -- fi_projection_set_profiling / fi_projection_read_profile
    def set_profiling(self, enable: bool) -> None:
        _check(self._lib.fi_projection_set_profiling(self._h, 1 if enable else 0))

    def read_profile(self):
        ms, n = ctypes.c_float(0.0), ctypes.c_int32(0)
        _check(self._lib.fi_projection_read_profile(self._h, ctypes.byref(ms), ctypes.byref(n)))
        return float(ms.value), int(n.value)

    # -- fi_projection_apply
    def apply(self, x: torch.Tensor, row_idx: Optional[torch.Tensor] = None, count: Optional[torch.Tensor] = None,
              out: Optional[torch.Tensor] = None) -> torch.Tensor:
        if x.dtype != torch.bfloat16 or x.dim() != 2 or x.shape[1] != self.in_dim or x.stride(1) != 1 or x.device != self.device:
            raise ValueError("x must be a bf16 [batch, in_dim] tensor on the projection's device with unit inner stride")
        batch = int(row_idx.numel()) if row_idx is not None else int(x.shape[0])
        if out is None:
            out = torch.zeros(batch, self.out_dim, dtype=torch.bfloat16, device=self.device)
        _check(self._lib.fi_projection_apply(self._h, _dp(x), x.stride(0), _dp(row_idx), batch, _dp(count), _dp(out),
                                             out.stride(0), _stream_ptr(self.device)))
        return out


def merge_shard_lookups(dist: torch.Tensor, global_idx: torch.Tensor, label: torch.Tensor, weight: torch.Tensor, *,
                        metric: int = FI_METRIC_SQL2, rule: int = FI_HIT_CONF_GT, threshold: float = 0.0) -> LookupOut:
    """fi_merge_shard_lookups on gathered tuples of shape [shards, batch, k]."""
    shards, batch, k = dist.shape
    out = LookupOut(batch, k, dist.device)
    st = out.as_struct()
    with torch.cuda.device(dist.device):
        _check(load_library().fi_merge_shard_lookups(shards, batch, k, _dp(dist.contiguous()), _dp(global_idx.contiguous()),
                                                     _dp(label.contiguous()), _dp(weight.contiguous()), metric, rule,
                                                     float(threshold), ctypes.byref(st), _stream_ptr(dist.device)))
    return out


class CascadeState:
    """Device arrays of a batch walking through the layers (torch owns the memory)."""

    def __init__(self, batch0: int, device):
        self.batch0 = batch0
        self.device = torch.device(device)
        self.idx = [torch.empty(max(batch0, 1), dtype=torch.int32, device=device) for _ in range(2)]
        self.count = [torch.zeros(1, dtype=torch.int32, device=device) for _ in range(2)]
        self.final_label = torch.empty(max(batch0, 1), dtype=torch.int32, device=device)
        self.exit_stage = torch.empty(max(batch0, 1), dtype=torch.int32, device=device)
        self.final_conf = torch.empty(max(batch0, 1), dtype=torch.float32, device=device)
        self.stage = 0

    def struct_for_stage(self, stage: int) -> fi_cascade_state_t:
        src, dst = (stage - 1) & 1, stage & 1
        active_idx = None if stage == 0 else _dp(self.idx[src])
        active_count = None if stage == 0 else _dp(self.count[src])
        return fi_cascade_state_t(active_idx, active_count, _dp(self.idx[dst]), _dp(self.count[dst]),
                                  _dp(self.final_label), _dp(self.exit_stage), _dp(self.final_conf), stage, self.batch0)

    def survivors(self, stage: int):
        """(ids, count) tensors alive after `stage` ran."""
        return self.idx[stage & 1], self.count[stage & 1]


def cascade_init(state: CascadeState, num_stages: int) -> None:
    st = state.struct_for_stage(0)
    _check(load_library().fi_cascade_init(ctypes.byref(st), num_stages, state.device.index or 0,
                                          _stream_ptr(state.device)))
    state.stage = 0


def cascade_step(cache: FreezeCache, stage_acts: torch.Tensor, state: CascadeState, stage: Optional[int] = None) -> None:
    cache._check_vecs(stage_acts)
    if stage is None:
        stage = state.stage
    st = state.struct_for_stage(stage)
    _check(load_library().fi_cascade_step(cache.handle, _dp(stage_acts), stage_acts.stride(0), ctypes.byref(st),
                                          _stream_ptr(cache.device)))
    state.stage = stage + 1


def cascade_step_projected(cache: FreezeCache, proj: Projection, stage_acts: torch.Tensor, state: CascadeState,
                           stage: Optional[int] = None) -> None:
    """fi_cascade_step_projected: project the survivors' activations, look them up, compact the misses."""
    if stage is None:
        stage = state.stage
    st = state.struct_for_stage(stage)
    _check(load_library().fi_cascade_step_projected(cache.handle, proj.handle, _dp(stage_acts), stage_acts.stride(0),
                                                    ctypes.byref(st), _stream_ptr(cache.device)))
    state.stage = stage + 1


def cascade_run_host(caches: Sequence[FreezeCache], acts_host: Sequence[torch.Tensor], final_label: torch.Tensor,
                     exit_stage: torch.Tensor, final_conf: torch.Tensor, arrivals: Optional[torch.Tensor] = None) -> None:
    """All stages with HOST activations and HOST outputs (copies inside, synchronises before returning)."""
    n = len(caches)
    batch0 = int(acts_host[0].shape[0])
    for t in list(acts_host) + [final_label, exit_stage, final_conf]:
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("host variant: tensors must be contiguous host tensors")
    hs = (ctypes.c_void_p * n)(*[c.handle.value for c in caches])
    ap = (ctypes.c_void_p * n)(*[a.data_ptr() for a in acts_host])
    _check(load_library().fi_cascade_run_host(hs, n, ap, batch0, _dp(final_label), _dp(exit_stage), _dp(final_conf),
                                              _dp(arrivals), _stream_ptr(caches[0].device)))
