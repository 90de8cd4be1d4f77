"""disco_select_policy runs on the host over statistics records in host memory, so it is checked here without a
GPU: against the oracle's selection and against the rule written out, on records with ties at every level."""
import ctypes as C

import numpy as np
import pytest

from oracle.binding import OracleStats, lib as orc_lib
from paper_2502_11417_b200.api import PolicyStats, select_policy, DiscoError, lib


def _records(rng, P):
    O = orc_lib()
    gs, os_, rows = (PolicyStats * P)(), (OracleStats * P)(), []
    for k in range(P):
        b_ttft = int(rng.choice([300, 310, 311]))            # tail TTFT by histogram bin
        b_tbt = int(rng.choice([410, 422, 430]))             # bins around 0.2 s .. 0.3 s
        mean = float(rng.choice([0.4, 0.5]))
        cost = float(rng.choice([10.0, 20.0, 30.0]))
        gs[k].bin_p99_ttft, gs[k].bin_p99_tbt, gs[k].mean_ttft_s, gs[k].total_cost = b_ttft, b_tbt, mean, cost
        e_ttft, e_tbt = O.orc_bin_lower_edge(b_ttft) * 1e-6, O.orc_bin_lower_edge(b_tbt) * 1e-6
        os_[k].p99_ttft_s, os_[k].p99_tbt_s, os_[k].mean_ttft_s, os_[k].total_cost = e_ttft, e_tbt, mean, cost
        rows.append((e_ttft, mean, cost, e_tbt))
    return gs, os_, rows


def _by_definition(rows, cap, slo):
    feas = [(r[0], r[1], r[2], k) for k, r in enumerate(rows) if r[2] <= cap and r[3] <= slo]
    if feas:
        return 0, min(feas)[3]
    return -4, min((r[2], k) for k, r in enumerate(rows))[1]


@pytest.mark.parametrize("seed", range(12))
def test_host_selection_against_the_oracle_and_the_rule(seed):
    rng = np.random.default_rng(seed)
    P = int(rng.integers(1, 40))
    gs, os_, rows = _records(rng, P)
    O = orc_lib()
    edges = sorted({r[3] for r in rows})
    slos = [0.1, 10.0] + edges + [float(np.nextafter(np.float32(e), np.float32(0))) for e in edges]
    for cap in (25.0, 5.0, 10.0, 100.0):
        for slo in slos:
            slo32 = float(np.float32(slo))
            best = C.c_int32(-1)
            rc = O.orc_select(C.cast(os_, C.c_void_p), P, cap, slo32, C.byref(best))
            got = select_policy(gs, cap, slo)
            assert got == (rc, best.value) == _by_definition(rows, cap, slo32), (cap, slo)


def test_host_selection_rejects_bad_arguments():
    gs = (PolicyStats * 2)()
    gs[0].bin_p99_tbt = 900                                   # not a bin
    with pytest.raises(DiscoError) as ei:
        select_policy(gs, 1.0, 1.0)
    assert ei.value.code == -1
    best = C.c_int32(0)
    assert lib().disco_select_policy(None, 2, 1.0, 1.0, C.byref(best)) == -1
    assert lib().disco_select_policy(C.cast(gs, C.c_void_p), 0, 1.0, 1.0, C.byref(best)) == -1
