"""Thin ctypes binding of libdisco's C ABI (argument marshalling only).

PyTorch is used for device memory (per-pair output tensors, device-resident
trace arrays) and for the current CUDA stream; every step of the evaluation
runs in the library's own kernels.  There is no CPU path: importing works
anywhere, but every call needs the built library and a CUDA device.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

from . import build as _build

NBINS = 864
SERVER_ONLY, DEVICE_ONLY, RACE = 0, 1, 2
EINVAL, ENOMEM, ECUDA, EINFEASIBLE = -1, -2, -3, -4


class DiscoError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"libdisco error {code}: {msg}")
        self.code = code


class ServerProfile(C.Structure):
    _fields_ = [("tbt_s", C.c_float), ("jitter", C.c_float), ("c_prefill", C.c_float), ("c_decode", C.c_float)]


class DeviceProfile(C.Structure):
    _fields_ = [("prefill_tps", C.c_float), ("ttft_intercept_s", C.c_float), ("decode_tps", C.c_float),
                ("jitter", C.c_float), ("c_prefill", C.c_float), ("c_decode", C.c_float), ("lam", C.c_float)]


class TraceDesc(C.Structure):
    _fields_ = [("n", C.c_uint64), ("prompt_len", C.c_void_p), ("output_len", C.c_void_p),
                ("server_ttft_s", C.c_void_p), ("server_profile", C.c_void_p), ("device_profile", C.c_void_p),
                ("servers", C.c_void_p), ("n_servers", C.c_uint32), ("devices", C.c_void_p),
                ("n_devices", C.c_uint32), ("arrays_on_device", C.c_uint32), ("first_index", C.c_uint64)]


class Policy(C.Structure):
    _fields_ = [("budget", C.c_float), ("alpha", C.c_float), ("mig_threshold", C.c_float), ("t_m_s", C.c_float),
                ("r_c", C.c_float), ("flags", C.c_uint32), ("expected_len", C.c_uint32), ("l_immediate", C.c_uint32)]


class PairOut(C.Structure):
    _fields_ = [("ttft_s", C.c_void_p), ("tbt_mean_s", C.c_void_p), ("tbt_max_s", C.c_void_p), ("cost", C.c_void_p),
                ("tok_server", C.c_void_p), ("tok_device", C.c_void_p), ("mig_at", C.c_void_p),
                ("delayed", C.c_void_p), ("decision", C.c_void_p)]


class PolicyStats(C.Structure):
    _fields_ = [("mean_ttft_s", C.c_double), ("total_cost", C.c_double),
                ("p50_ttft_s", C.c_float), ("p95_ttft_s", C.c_float), ("p99_ttft_s", C.c_float),
                ("p99_tbt_s", C.c_float),
                ("bin_p50_ttft", C.c_int32), ("bin_p95_ttft", C.c_int32), ("bin_p99_ttft", C.c_int32),
                ("bin_p99_tbt", C.c_int32),
                ("n_requests", C.c_uint64), ("n_intervals", C.c_uint64),
                ("n_server_only", C.c_uint64), ("n_device_only", C.c_uint64), ("n_race", C.c_uint64),
                ("n_device_started", C.c_uint64), ("n_device_won", C.c_uint64), ("n_migrations", C.c_uint64),
                ("tok_server", C.c_uint64), ("tok_device", C.c_uint64),
                ("prefill_tok_server", C.c_uint64), ("prefill_tok_device", C.c_uint64),
                ("delayed_tokens", C.c_uint64)]


class Prep(C.Structure):
    _fields_ = [("device_constrained", C.c_int32), ("l_th", C.c_int32), ("l_star", C.c_int32), ("B", C.c_int32),
                ("w_star", C.c_int64), ("w_tail", C.c_int64), ("tau", C.c_int64),
                ("beta_rule", C.c_int32), ("l_immediate", C.c_int32), ("beta", C.c_int64)]


EXPORTS = ["disco_load_trace", "disco_eval_policies", "disco_reduce_stats", "disco_select_policy",
           "disco_get_histograms", "disco_get_prep", "disco_get_group_tables", "disco_free_trace",
           "disco_last_error", "disco_set_timing", "disco_get_timing", "disco_kernel_launch_count",
           "disco_sort_ttft_ticks_noalloc", "disco_select_policy_device", "disco_set_group_tables",
           "disco_accumulator_words", "disco_export_accumulators", "disco_import_accumulators",
           "disco_measure_alu_peak", "disco_get_work_counts", "disco_debug_selftest"]

PAIR_FIELDS = [("ttft_s", "float32"), ("tbt_mean_s", "float32"), ("tbt_max_s", "float32"), ("cost", "float32"),
               ("tok_server", "uint32"), ("tok_device", "uint32"), ("mig_at", "uint32"), ("delayed", "uint16"),
               ("decision", "uint8")]

_lib = None


def library_path() -> str:
    return _build.LIB


def lib() -> C.CDLL:
    """Loads libdisco.so (building it first if the sources are newer).  Raises if it cannot be had.  With
    DISCO_CHECKED_BUILD=1 in the environment the index-checking variant (-DDISCO_DEBUG) is built and loaded instead."""
    global _lib
    if _lib is None:
        path = _build.build(checked=os.environ.get("DISCO_CHECKED_BUILD") == "1")
        L = C.CDLL(path)
        vp, u32, u64 = C.c_void_p, C.c_uint32, C.c_uint64
        L.disco_load_trace.restype = C.c_int; L.disco_load_trace.argtypes = [C.POINTER(vp), vp, vp]
        L.disco_eval_policies.restype = C.c_int; L.disco_eval_policies.argtypes = [vp, vp, u32, u64, vp, vp]
        L.disco_reduce_stats.restype = C.c_int; L.disco_reduce_stats.argtypes = [vp, vp, vp]
        L.disco_select_policy.restype = C.c_int
        L.disco_select_policy.argtypes = [vp, u32, C.c_double, C.c_float, C.POINTER(C.c_int32)]
        L.disco_select_policy_device.restype = C.c_int
        L.disco_select_policy_device.argtypes = [vp, C.c_double, C.c_float, C.POINTER(C.c_int32), vp]
        L.disco_set_group_tables.restype = C.c_int; L.disco_set_group_tables.argtypes = [vp, vp, vp, vp, vp]
        L.disco_accumulator_words.restype = u64; L.disco_accumulator_words.argtypes = [vp]
        L.disco_export_accumulators.restype = C.c_int; L.disco_export_accumulators.argtypes = [vp, vp, vp]
        L.disco_import_accumulators.restype = C.c_int; L.disco_import_accumulators.argtypes = [vp, vp, vp]
        L.disco_get_work_counts.restype = C.c_int; L.disco_get_work_counts.argtypes = [vp, vp, vp]
        L.disco_debug_selftest.restype = C.c_int; L.disco_debug_selftest.argtypes = [vp]
        L.disco_measure_alu_peak.restype = C.c_int
        L.disco_measure_alu_peak.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), vp]
        L.disco_get_histograms.restype = C.c_int; L.disco_get_histograms.argtypes = [vp, u32, vp, vp, vp]
        L.disco_get_prep.restype = C.c_int; L.disco_get_prep.argtypes = [vp, u32, u32, vp, vp]
        L.disco_get_group_tables.restype = C.c_int64
        L.disco_get_group_tables.argtypes = [vp, u32, vp, vp, vp, u64, vp]
        L.disco_free_trace.restype = None; L.disco_free_trace.argtypes = [vp]
        L.disco_last_error.restype = C.c_char_p
        L.disco_set_timing.restype = C.c_int; L.disco_set_timing.argtypes = [vp, C.c_int]
        L.disco_get_timing.restype = C.c_int
        L.disco_get_timing.argtypes = [vp, C.POINTER(C.c_float)]
        L.disco_kernel_launch_count.restype = u64; L.disco_kernel_launch_count.argtypes = []
        L.disco_sort_ttft_ticks_noalloc.restype = C.c_int
        L.disco_sort_ttft_ticks_noalloc.argtypes = [vp, u32, vp, vp]
        _lib = L
    return _lib


def kernel_launch_count() -> int:
    return int(lib().disco_kernel_launch_count())


def _check(rc: int, allow=()):
    if rc != 0 and rc not in allow:
        raise DiscoError(rc, lib().disco_last_error().decode())
    return rc


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


_cuda_ok = None


def _require_cuda():
    global _cuda_ok
    if _cuda_ok is None:
        import torch
        _cuda_ok = bool(torch.cuda.is_available())
    if not _cuda_ok:
        raise DiscoError(ECUDA, "no CUDA device: libdisco has no CPU path")


_stats_dtype = None


def stats_view(stats):
    """The (PolicyStats * P) array returned by reduce_stats as a numpy structured array (no copy), for
    column-wise reads such as stats_view(st)["total_cost"].min()."""
    global _stats_dtype
    if _stats_dtype is None:
        _stats_dtype = np.dtype(PolicyStats)
    return np.frombuffer(stats, dtype=_stats_dtype)


def _torch_dtype(name):
    import torch
    return getattr(torch, name)


def server_array(servers: Sequence[Dict[str, float]]):
    arr = (ServerProfile * len(servers))()
    for k, s in enumerate(servers):
        arr[k] = ServerProfile(s["tbt_s"], s["jitter"], s["c_prefill"], s["c_decode"])
    return arr


def device_array(devices: Sequence[Dict[str, float]]):
    arr = (DeviceProfile * len(devices))()
    for k, d in enumerate(devices):
        arr[k] = DeviceProfile(d["prefill_tps"], d["ttft_intercept_s"], d["decode_tps"], d["jitter"],
                               d["c_prefill"], d["c_decode"], d["lam"])
    return arr


def policy_array(policies: Sequence[Dict[str, float]]):
    arr = (Policy * len(policies))()
    for k, p in enumerate(policies):
        arr[k] = Policy(p["budget"], p["alpha"], p["mig_threshold"], p["t_m_s"], p["r_c"], p["flags"],
                        p.get("expected_len", 0), p.get("l_immediate", 0))
    return arr


def select_policy(stats, cost_cap: float, tbt_slo_s: float):
    """disco_select_policy over a (PolicyStats * P) array in host memory (the records of reduce_stats, or
    merged ones).  Returns (status, index): status 0, or EINFEASIBLE with the cheapest policy's index."""
    best = C.c_int32(-1)
    rc = _check(lib().disco_select_policy(C.cast(stats, C.c_void_p), len(stats), cost_cap, tbt_slo_s, C.byref(best)),
                allow=(EINFEASIBLE,))
    return rc, best.value


def measure_alu_peak(stream=None):
    """disco_measure_alu_peak: (lane-instructions/s, token-steps/s) the GPU sustains on the token loop's
    instruction mix."""
    _require_cuda()
    a, b = C.c_double(0.0), C.c_double(0.0)
    _check(lib().disco_measure_alu_peak(C.byref(a), C.byref(b), _stream_ptr(stream)))
    return a.value, b.value


NOALLOC_MAX_N = 262144


def sort_ttft_ticks_noalloc(server_ttft_s, sorted_ticks, stream=None):
    """disco_sort_ttft_ticks_noalloc: server_ttft_s is a CUDA float32 tensor [n], sorted_ticks a CUDA int32
    tensor [n] that receives the ascending microsecond ticks.  The library allocates nothing in this call;
    both tensors are the caller's.  Calls on one GPU must not overlap (they share one working array)."""
    import torch
    for t, dt in ((server_ttft_s, torch.float32), (sorted_ticks, torch.int32)):
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dt and t.is_contiguous() and t.dim() == 1):
            raise ValueError("expected contiguous 1-D CUDA tensors: float32 in, int32 out")
    if server_ttft_s.numel() != sorted_ticks.numel():
        raise ValueError("input and output lengths differ")
    n = server_ttft_s.numel()
    if n >= 1 << 32:
        raise ValueError("too many requests")
    _check(lib().disco_sort_ttft_ticks_noalloc(server_ttft_s.data_ptr() if n else None, n,
                                               sorted_ticks.data_ptr() if n else None, _stream_ptr(stream)))
    return sorted_ticks


class Trace:
    """A trace loaded on the GPU (wraps disco_ctx_t).  Methods mirror the C entry points."""

    def __init__(self):
        self._h = C.c_void_p(None)
        self.n = 0
        self.P = 0
        self._keep = None

    # -- disco_load_trace ---------------------------------------------------------------------------------
    def load_trace(self, prompt_len, output_len, server_ttft_s, server_profile, device_profile, servers, devices,
                   stream=None, first_index: int = 0, staged_copy: bool = False):
        """Arrays may be numpy arrays / pinned CPU tensors (host memory) or CUDA tensors (device memory),
        all of the same kind.  Reloading reuses the context's device memory.  first_index: position of these
        arrays' first request in the whole trace when they are a shard of it.  staged_copy: host arrays are copied
        by the copy engine even when they are page-locked (instead of being read in place by the ingestion kernel)."""
        import torch
        _require_cuda()
        arrs = [prompt_len, output_len, server_ttft_s, server_profile, device_profile]
        on_dev = isinstance(prompt_len, torch.Tensor) and prompt_len.is_cuda
        want = [("int32", np.int32), ("int32", np.int32), ("float32", np.float32), ("uint8", np.uint8),
                ("uint8", np.uint8)]
        ptrs, keep = [], []
        for a, (tname, npdt) in zip(arrs, want):
            if a is None:
                ptrs.append(None)
                continue
            if isinstance(a, torch.Tensor):
                if a.is_cuda != on_dev:
                    raise ValueError("all trace arrays must live on the same side")
                t = a.contiguous()
                if t.dtype != _torch_dtype(tname):
                    raise TypeError(f"expected {tname}, got {t.dtype}")
                keep.append(t)
                ptrs.append(t.data_ptr())
            else:
                if on_dev:
                    raise ValueError("all trace arrays must live on the same side")
                x = np.ascontiguousarray(a, dtype=npdt)
                keep.append(x)
                ptrs.append(x.ctypes.data)
        n = int(len(prompt_len))
        sv, dv = server_array(servers), device_array(devices)
        desc = TraceDesc(n, ptrs[0], ptrs[1], ptrs[2], ptrs[3], ptrs[4], C.cast(sv, C.c_void_p), len(servers),
                         C.cast(dv, C.c_void_p), len(devices), 1 if on_dev else (2 if staged_copy else 0),
                         int(first_index))
        _check(lib().disco_load_trace(C.byref(self._h), C.byref(desc), _stream_ptr(stream)))
        self.n = n
        self.n_groups = len(servers) * len(devices)
        return self

    @classmethod
    def from_workload(cls, w, stream=None) -> "Trace":
        return cls().load_trace(w.prompt_len, w.output_len, w.server_ttft_s, w.server_profile, w.device_profile,
                                w.servers, w.devices, stream=stream)

    # -- disco_eval_policies -------------------------------------------------------------------------------
    def alloc_pair_outputs(self, P: int, fields: Optional[Sequence[str]] = None):
        import torch
        fields = [f for f, _ in PAIR_FIELDS] if fields is None else list(fields)
        return {f: torch.empty((P, self.n), dtype=_torch_dtype(dt), device="cuda")
                for f, dt in PAIR_FIELDS if f in fields}

    def eval_policies(self, policies, seed: int, out: Optional[Dict[str, "object"]] = None, stream=None):
        """policies: list of dicts or a prepared (Policy * P) array.  out: dict of CUDA tensors [P, n]."""
        arr = policies if isinstance(policies, C.Array) else policy_array(policies)
        P = len(arr)
        po = None
        if out is not None:
            vals = {}
            for f, dt in PAIR_FIELDS:
                t = out.get(f)
                if t is not None:
                    if not t.is_cuda or t.dtype != _torch_dtype(dt) or tuple(t.shape) != (P, self.n) \
                            or not t.is_contiguous():
                        raise ValueError(f"output '{f}' must be a contiguous CUDA tensor [P, n] of {dt}")
                    vals[f] = t.data_ptr()
            po = PairOut(*[vals.get(f) for f, _ in PAIR_FIELDS])
        _check(lib().disco_eval_policies(self._h, C.cast(arr, C.c_void_p), P, seed,
                                         C.byref(po) if po is not None else None, _stream_ptr(stream)))
        self.P = P
        self._keep = (arr, out)
        return self

    # -- disco_reduce_stats --------------------------------------------------------------------------------
    def reduce_stats(self, stream=None):
        stats = (PolicyStats * self.P)()
        _check(lib().disco_reduce_stats(self._h, C.cast(stats, C.c_void_p), _stream_ptr(stream)))
        return stats

    # -- disco_select_policy -------------------------------------------------------------------------------
    def select_policy(self, cost_cap: float, tbt_slo_s: float, stream=None):
        """disco_select_policy_device: the selection by a kernel over the records of the last reduce_stats.
        Returns (status, index): status 0, or EINFEASIBLE with the cheapest policy's index."""
        best = C.c_int32(-1)
        rc = _check(lib().disco_select_policy_device(self._h, cost_cap, tbt_slo_s, C.byref(best),
                                                     _stream_ptr(stream)), allow=(EINFEASIBLE,))
        return rc, best.value

    # -- shards of one trace ---------------------------------------------------------------------------------
    def set_group_tables(self, cnt, ticks, n_ticks, stream=None):
        """disco_set_group_tables: cnt int64 [G, 4097] and n_ticks uint64 [G] as numpy arrays; ticks int32, the
        groups one after the other in any order within a group, a numpy array or a CUDA tensor."""
        cnt = np.ascontiguousarray(cnt, dtype=np.int64)
        ns = np.ascontiguousarray(n_ticks, dtype=np.uint64)
        if isinstance(ticks, np.ndarray):
            ticks = np.ascontiguousarray(ticks, dtype=np.int32)
            ptr, size = ticks.ctypes.data, ticks.size
        else:
            if ticks.dtype != _torch_dtype("int32") or not ticks.is_contiguous():
                raise TypeError("ticks must be a contiguous int32 tensor")
            ptr, size = ticks.data_ptr(), ticks.numel()
        if cnt.shape != (self.n_groups, 4097) or ns.shape != (self.n_groups,) or size != int(ns.sum()):
            raise ValueError("cnt must be [G, 4097], n_ticks [G], ticks of their total length")
        _check(lib().disco_set_group_tables(self._h, cnt.ctypes.data, ptr if size else None, ns.ctypes.data,
                                            _stream_ptr(stream)))
        return self

    def accumulator_words(self) -> int:
        return int(lib().disco_accumulator_words(self._h))

    def export_accumulators(self, out=None, stream=None):
        """The additive accumulator words of the last evaluation: a numpy uint64 array (host), or written into
        `out`, a CUDA int64 / numpy uint64 buffer of accumulator_words() elements."""
        k = self.accumulator_words()
        if out is None:
            out = np.zeros(k, dtype=np.uint64)
        if isinstance(out, np.ndarray):
            ptr, size, width = out.ctypes.data, out.size, out.dtype.itemsize
        else:
            ptr, size, width = out.data_ptr(), out.numel(), out.element_size()
        if size != k or width != 8:
            raise ValueError("accumulator buffer must hold accumulator_words() 64-bit words")
        _check(lib().disco_export_accumulators(self._h, ptr, _stream_ptr(stream)))
        return out

    def import_accumulators(self, words, stream=None):
        k = self.accumulator_words()
        if isinstance(words, np.ndarray):
            words = np.ascontiguousarray(words, dtype=np.uint64)
            ptr, size = words.ctypes.data, words.size
        else:
            ptr, size = words.data_ptr(), words.numel()
        if size != k:
            raise ValueError("accumulator buffer must hold accumulator_words() 64-bit words")
        _check(lib().disco_import_accumulators(self._h, ptr, _stream_ptr(stream)))
        return self

    # -- inspection ----------------------------------------------------------------------------------------
    def histograms(self, p: int, stream=None):
        a = np.zeros(NBINS, dtype=np.uint64)
        b = np.zeros(NBINS, dtype=np.uint64)
        _check(lib().disco_get_histograms(self._h, p, a.ctypes.data, b.ctypes.data, _stream_ptr(stream)))
        return a, b

    def prep(self, g: int, p: int, stream=None) -> Prep:
        out = Prep()
        _check(lib().disco_get_prep(self._h, g, p, C.byref(out), _stream_ptr(stream)))
        return out

    def group_size(self, g: int, stream=None) -> int:
        """Requests of profile group g in the loaded trace."""
        ng = lib().disco_get_group_tables(self._h, g, None, None, None, 0, _stream_ptr(stream))
        if ng < 0:
            _check(int(ng))
        return int(ng)

    def group_tables(self, g: int, n_sorted: Optional[int] = None, stream=None):
        cnt = np.zeros(4097, dtype=np.int64)
        kn = np.zeros(257, dtype=np.int32)
        ng = lib().disco_get_group_tables(self._h, g, None, None, None, 0, _stream_ptr(stream))
        if ng < 0:
            _check(int(ng))
        k = int(ng) if n_sorted is None else min(int(ng), n_sorted)
        srt = np.zeros(max(k, 1), dtype=np.int32)
        rc = lib().disco_get_group_tables(self._h, g, cnt.ctypes.data, kn.ctypes.data, srt.ctypes.data, k,
                                          _stream_ptr(stream))
        if rc < 0:
            _check(int(rc))
        return cnt, kn, srt[:k]

    def sorted_ticks_device(self, g: int, stream=None):
        """Group g's ascending server-TTFT ticks as a CUDA int32 tensor (a device-to-device copy)."""
        import torch
        ng = lib().disco_get_group_tables(self._h, g, None, None, None, 0, _stream_ptr(stream))
        if ng < 0:
            _check(int(ng))
        out = torch.empty(int(ng), dtype=torch.int32, device="cuda")
        if ng:
            rc = lib().disco_get_group_tables(self._h, g, None, None, out.data_ptr(), int(ng), _stream_ptr(stream))
            if rc < 0:
                _check(int(rc))
        return out

    def set_timing(self, on: bool = True):
        _check(lib().disco_set_timing(self._h, int(on)))

    def timing(self):
        """Device milliseconds of the last reduced evaluation's kernels:
        (clamp-free play-out, general play-out, pair reductions, per-pair rows)."""
        ms = (C.c_float * 4)()
        _check(lib().disco_get_timing(self._h, ms))
        return tuple(ms)

    def work_counts(self, stream=None):
        """(pairs settled zone by zone, pairs evaluated one by one, requests settled per policy family, sweeps
        over chunk segments) of the last evaluation."""
        w = (C.c_uint64 * 4)()
        _check(lib().disco_get_work_counts(self._h, w, _stream_ptr(stream)))
        return tuple(int(x) for x in w)

    def close(self):
        if self._h:
            lib().disco_free_trace(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
