"""ctypes binding of the CPU oracle (test infrastructure only)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "disco_oracle.cpp")
_HDR = os.path.join(_HERE, "disco_oracle.h")
_SO = os.path.join(_HERE, "liborc_disco.so")

NBINS = 864
SERVER_ONLY, DEVICE_ONLY, RACE = 0, 1, 2


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with g++ (FP contraction off) if the library is stale."""
    stale = force or not os.path.exists(_SO) or os.path.getmtime(_SO) < max(
        os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if stale:
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared",
                               "-Wall", "-Wextra", "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


class server_struct(C.Structure):
    _fields_ = [("tbt_s", C.c_float), ("jitter", C.c_float), ("c_prefill", C.c_float), ("c_decode", C.c_float)]


class device_struct(C.Structure):
    _fields_ = [("prefill_tps", C.c_float), ("ttft_intercept_s", C.c_float), ("decode_tps", C.c_float),
                ("jitter", C.c_float), ("c_prefill", C.c_float), ("c_decode", C.c_float), ("lam", C.c_float)]


class policy_struct(C.Structure):
    _fields_ = [("budget", C.c_float), ("alpha", C.c_float), ("mig_threshold", C.c_float),
                ("t_m_s", C.c_float), ("r_c", C.c_float), ("flags", C.c_uint32), ("expected_len", C.c_uint32),
                ("l_immediate", C.c_uint32)]


class prep_struct(C.Structure):
    _fields_ = [("device_constrained", C.c_int32), ("l_th", C.c_int32), ("l_star", C.c_int32), ("B", C.c_int32),
                ("w_star", C.c_int64), ("w_tail", C.c_int64), ("tau", C.c_int64), ("t_m", C.c_int64),
                ("candidate_winner", C.c_int32), ("delta_c", C.c_float),
                ("funded_fraction", C.c_double), ("budget_A", C.c_double),
                ("beta_rule", C.c_int32), ("l_immediate", C.c_int32), ("beta", C.c_int64)]


class pair_out_struct(C.Structure):
    _fields_ = [("ttft_s", C.c_void_p), ("tbt_mean_s", C.c_void_p), ("tbt_max_s", C.c_void_p), ("cost", C.c_void_p),
                ("tok_server", C.c_void_p), ("tok_device", C.c_void_p), ("mig_at", C.c_void_p),
                ("delayed", C.c_void_p), ("decision", C.c_void_p)]


class OracleStats(C.Structure):
    _fields_ = [("n_requests", C.c_uint64), ("n_intervals", C.c_uint64),
                ("sum_ttft_s", C.c_double), ("total_cost", C.c_double),
                ("n_server_only", C.c_uint64), ("n_device_only", C.c_uint64), ("n_race", C.c_uint64),
                ("n_device_started", C.c_uint64), ("n_device_won", C.c_uint64), ("n_migrations", C.c_uint64),
                ("tok_server", C.c_uint64), ("tok_device", C.c_uint64),
                ("prefill_tok_server", C.c_uint64), ("prefill_tok_device", C.c_uint64),
                ("delayed_tokens", C.c_uint64),
                ("ttft_hist", C.c_uint64 * NBINS), ("tbt_hist", C.c_uint64 * NBINS),
                ("mean_ttft_s", C.c_double),
                ("p50_ttft_s", C.c_double), ("p95_ttft_s", C.c_double), ("p99_ttft_s", C.c_double),
                ("p99_tbt_s", C.c_double),
                ("bin_p50_ttft", C.c_int32), ("bin_p95_ttft", C.c_int32), ("bin_p99_ttft", C.c_int32),
                ("bin_p99_tbt", C.c_int32),
                ("exact_p50_ttft_s", C.c_double), ("exact_p95_ttft_s", C.c_double),
                ("exact_p99_ttft_s", C.c_double), ("exact_p99_tbt_s", C.c_double)]


ADDITIVE_FIELDS = ["n_requests", "n_intervals", "sum_ttft_s", "total_cost", "n_server_only", "n_device_only",
                   "n_race", "n_device_started", "n_device_won", "n_migrations", "tok_server", "tok_device",
                   "prefill_tok_server", "prefill_tok_device", "delayed_tokens"]

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        # DISCO_ORACLE_LIB: a library built elsewhere from a deliberately broken copy of the source (the mutation
        # check of the pins, tests/oracle_mutants.py).  It is honoured only together with the marker that script
        # sets, so that a stray variable cannot swap the checker under an ordinary test run.
        swapped = os.environ.get("DISCO_ORACLE_LIB")
        if swapped and os.environ.get("DISCO_ORACLE_MUTATION_CHECK") != "1":
            raise RuntimeError("DISCO_ORACLE_LIB is set outside the mutation check (tests/oracle_mutants.py)")
        L = C.CDLL(swapped or build_oracle())
        L.orc_mix.restype = C.c_uint32; L.orc_mix.argtypes = [C.c_uint32]
        L.orc_hash.restype = C.c_uint32; L.orc_hash.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32]
        L.orc_jitter.restype = C.c_int64; L.orc_jitter.argtypes = [C.c_uint32, C.c_int64]
        L.orc_bin.restype = C.c_int32; L.orc_bin.argtypes = [C.c_int64]
        L.orc_bin_lower_edge.restype = C.c_int64; L.orc_bin_lower_edge.argtypes = [C.c_int32]
        L.orc_seconds_to_ticks.restype = C.c_int64; L.orc_seconds_to_ticks.argtypes = [C.c_float]
        L.orc_rate_to_ticks.restype = C.c_int64; L.orc_rate_to_ticks.argtypes = [C.c_float]
        L.orc_last_error.restype = C.c_char_p
        L.orc_load.restype = C.c_void_p
        L.orc_load.argtypes = [C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                               C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32]
        L.orc_free.argtypes = [C.c_void_p]
        L.orc_n_groups.restype = C.c_uint32; L.orc_n_groups.argtypes = [C.c_void_p]
        L.orc_group_tables.restype = C.c_int64
        L.orc_group_tables.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_inverse_cdf.restype = C.c_int64; L.orc_inverse_cdf.argtypes = [C.c_void_p, C.c_uint32, C.c_double]
        L.orc_prep.restype = C.c_int
        L.orc_prep.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]
        L.orc_play.restype = C.c_int
        L.orc_play.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p,
                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_eval.restype = C.c_int
        L.orc_eval.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64,
                               C.c_void_p, C.c_void_p, C.c_int]
        L.orc_eval_cols.restype = C.c_int
        L.orc_eval_cols.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64,
                                    C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_int]
        L.orc_finish.argtypes = [C.c_void_p, C.c_uint32]
        L.orc_select.restype = C.c_int
        L.orc_select.argtypes = [C.c_void_p, C.c_uint32, C.c_double, C.c_double, C.c_void_p]
        _lib = L
    return _lib


def _servers(servers: Sequence[Dict[str, float]]):
    arr = (server_struct * len(servers))()
    for k, s in enumerate(servers):
        arr[k] = server_struct(s["tbt_s"], s["jitter"], s["c_prefill"], s["c_decode"])
    return arr


def _devices(devices: Sequence[Dict[str, float]]):
    arr = (device_struct * len(devices))()
    for k, d in enumerate(devices):
        arr[k] = device_struct(d["prefill_tps"], d["ttft_intercept_s"], d["decode_tps"], d["jitter"],
                               d["c_prefill"], d["c_decode"], d["lam"])
    return arr


def _policies(policies: Sequence[Dict[str, float]]):
    arr = (policy_struct * len(policies))()
    for k, p in enumerate(policies):
        arr[k] = policy_struct(p["budget"], p["alpha"], p["mig_threshold"], p["t_m_s"], p["r_c"], p["flags"],
                               p.get("expected_len", 0), p.get("l_immediate", 0))
    return arr


_PAIR_FIELDS = [("ttft_s", np.float64), ("tbt_mean_s", np.float64), ("tbt_max_s", np.float64),
                ("cost", np.float64), ("tok_server", np.uint32), ("tok_device", np.uint32),
                ("mig_at", np.uint32), ("delayed", np.uint16), ("decision", np.uint8)]


class Oracle:
    """A loaded trace on the CPU oracle."""

    def __init__(self, prompt_len, output_len, server_ttft_s, server_profile, device_profile, servers, devices):
        self.L = lib()
        self.n = int(len(prompt_len))
        self._pl = np.ascontiguousarray(prompt_len, dtype=np.int32)
        self._ol = np.ascontiguousarray(output_len, dtype=np.int32)
        self._tt = np.ascontiguousarray(server_ttft_s, dtype=np.float32)
        self._sp = None if server_profile is None else np.ascontiguousarray(server_profile, dtype=np.uint8)
        self._dp = None if device_profile is None else np.ascontiguousarray(device_profile, dtype=np.uint8)
        sv, dv = _servers(servers), _devices(devices)
        self.h = self.L.orc_load(self.n, self._pl.ctypes.data, self._ol.ctypes.data, self._tt.ctypes.data,
                                 None if self._sp is None else self._sp.ctypes.data,
                                 None if self._dp is None else self._dp.ctypes.data,
                                 C.cast(sv, C.c_void_p), len(servers), C.cast(dv, C.c_void_p), len(devices))
        if not self.h:
            raise ValueError(self.L.orc_last_error().decode())

    @classmethod
    def from_workload(cls, w) -> "Oracle":
        return cls(w.prompt_len, w.output_len, w.server_ttft_s, w.server_profile, w.device_profile,
                   w.servers, w.devices)

    def close(self):
        if self.h:
            self.L.orc_free(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def n_groups(self) -> int:
        return int(self.L.orc_n_groups(self.h))

    def group_tables(self, g: int):
        ng = self.L.orc_group_tables(self.h, g, None, None, None)
        cnt = np.zeros(4097, dtype=np.int64)
        srt = np.zeros(max(int(ng), 1), dtype=np.int64)
        kn = np.zeros(257, dtype=np.int64)
        self.L.orc_group_tables(self.h, g, cnt.ctypes.data, srt.ctypes.data, kn.ctypes.data)
        return cnt, srt[:ng], kn

    def inverse_cdf(self, g: int, q: float) -> int:
        return int(self.L.orc_inverse_cdf(self.h, g, q))

    def prep(self, policy: Dict[str, float], g: int = 0) -> prep_struct:
        arr = _policies([policy])
        out = prep_struct()
        if self.L.orc_prep(self.h, C.cast(arr, C.c_void_p), g, C.byref(out)) != 0:
            raise ValueError(self.L.orc_last_error().decode())
        return out

    def play(self, policy: Dict[str, float], seed: int, i: int):
        n = int(self._ol[i])
        g = np.zeros(n + 1, dtype=np.int64)
        d = np.zeros(n + 1, dtype=np.int64)
        ttft = C.c_int64(); wd = C.c_int32(); mig = C.c_int32(); lat = C.c_int64(); dl = C.c_int32()
        arr = _policies([policy])
        dec = self.L.orc_play(self.h, C.cast(arr, C.c_void_p), seed, i, g.ctypes.data, d.ctypes.data,
                              C.byref(ttft), C.byref(wd), C.byref(mig), C.byref(lat), C.byref(dl))
        if dec < 0:
            raise ValueError(self.L.orc_last_error().decode())
        return dict(decision=dec, g=g, d=d, ttft=ttft.value, winner_is_device=bool(wd.value), mig_at=mig.value,
                    mig_latency=lat.value, delayed=dl.value)

    def eval(self, policies: Sequence[Dict[str, float]], seed: int, i0: int = 0, i1: Optional[int] = None,
             pairs: bool = False, exact: bool = False, finish: bool = True):
        """Returns (stats array, per-pair dict or None)."""
        i1 = self.n if i1 is None else i1
        P = len(policies)
        arr = _policies(policies)
        stats = (OracleStats * P)()
        out = None
        po = None
        if pairs:
            out = {name: np.zeros((P, self.n), dtype=dt) for name, dt in _PAIR_FIELDS}
            po = pair_out_struct(*[out[name].ctypes.data for name, _ in _PAIR_FIELDS])
        rc = self.L.orc_eval(self.h, C.cast(arr, C.c_void_p), P, seed, i0, i1,
                             C.byref(po) if po is not None else None, C.cast(stats, C.c_void_p), int(exact))
        if rc != 0:
            raise ValueError(self.L.orc_last_error().decode())
        if finish:
            self.L.orc_finish(C.cast(stats, C.c_void_p), P)
        return stats, out

    def eval_columns(self, policies: Sequence[Dict[str, float]], seed: int, ranges):
        """Per-pair results of the requests in `ranges` (a list of (i0, i1)) only: a dict of arrays [P, K], K the
        total length of the ranges, columns in the order of the ranges.  Memory is O(P K), whatever the trace's
        size."""
        P = len(policies)
        K = sum(i1 - i0 for i0, i1 in ranges)
        arr = _policies(policies)
        out = {name: np.zeros((P, K), dtype=dt) for name, dt in _PAIR_FIELDS}
        stats = (OracleStats * P)()
        col = 0
        for i0, i1 in ranges:
            po = pair_out_struct(*[out[name].ctypes.data + col * out[name].itemsize for name, _ in _PAIR_FIELDS])
            rc = self.L.orc_eval_cols(self.h, C.cast(arr, C.c_void_p), P, seed, i0, i1, C.byref(po), K, i0,
                                      C.cast(stats, C.c_void_p), 0)
            if rc != 0:
                raise ValueError(self.L.orc_last_error().decode())
            col += i1 - i0
        return out

    def finish(self, stats):
        self.L.orc_finish(C.cast(stats, C.c_void_p), len(stats))

    def select(self, stats, cost_cap: float, tbt_slo_s: float):
        best = C.c_int32(-1)
        rc = self.L.orc_select(C.cast(stats, C.c_void_p), len(stats), cost_cap, tbt_slo_s, C.byref(best))
        return rc, best.value


def merge_stats(parts: List) -> "C.Array":
    """Sum the additive fields and histograms of several stats arrays (disjoint request ranges)."""
    P = len(parts[0])
    tot = (OracleStats * P)()
    for part in parts:
        for p in range(P):
            for f in ADDITIVE_FIELDS:
                setattr(tot[p], f, getattr(tot[p], f) + getattr(part[p], f))
            a = np.ctypeslib.as_array(tot[p].ttft_hist); a += np.ctypeslib.as_array(part[p].ttft_hist)
            b = np.ctypeslib.as_array(tot[p].tbt_hist); b += np.ctypeslib.as_array(part[p].tbt_hist)
    return tot
