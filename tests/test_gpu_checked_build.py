"""The checked build (-DDISCO_DEBUG): the same kernels with every derived index tested against its bound before the
access.  The tiny and edge-case parity cases must run through it with no index refused and still match the oracle;
and the checks must be live (needs a GPU).  Each part runs in a process of its own, because a process loads either
the ordinary or the checked library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CASES = ("test_config0_full or test_config1_shape or test_config3_shape or test_config4_shape or test_config5_shape "
         "or test_edge_cases or test_empty_trace or test_flag_and_mode_matrix or test_buffer_search_paths "
         "or test_stochastic_baselines or test_linear_wait_rule or test_zone_by_zone or test_more_than_32_policy_tiles "
         "or test_mixed_timeline_classes or test_generation_slower or test_sorted_ticks_around "
         "or test_one_prompt_length or test_more_groups_than_fit or test_family_whose_first_tile")


def _run(args):
    env = dict(os.environ, DISCO_CHECKED_BUILD="1")
    return subprocess.run([sys.executable] + args, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)


def test_parity_cases_pass_with_every_index_checked():
    r = _run(["-m", "pytest", "tests/test_gpu_parity.py", "tests/test_gpu_shards.py", "tests/test_zz_no_alloc.py",
              "-x", "-q", "-m", "gpu", "-k", CASES + " or shards or two_calls or limits"])
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout


def test_the_checks_are_live():
    code = (
        "import ctypes\n"
        "from paper_2502_11417_b200 import api, synth, Trace\n"
        "L = api.lib()\n"
        "assert api._build.LIB_CHECKED in [api._build.build(checked=True)]\n"
        "rc = L.disco_debug_selftest(None)\n"
        "msg = L.disco_last_error().decode()\n"
        "assert rc == -3 and 'checked build' in msg and 'self-test' in msg and 'index 34' in msg and 'bound 32' in msg, (rc, msg)\n"
        "assert L.disco_debug_selftest(None) == -3\n"              # the record is cleared and taken again
        "w = synth.make_workload(1, n=3000, n_budgets=5)\n"          # the context is still usable after a refusal
        "t = Trace.from_workload(w); t.eval_policies(w.policies, 1); s = t.reduce_stats()\n"
        "assert s[0].n_requests == 3000\n"
        "print('live')\n")
    r = _run(["-c", code])
    assert r.returncode == 0 and "live" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


def test_the_ordinary_build_has_no_selftest():
    from paper_2502_11417_b200 import api
    if os.environ.get("DISCO_CHECKED_BUILD") == "1":
        pytest.skip("this process runs the checked build")
    L = api.lib()
    assert L.disco_debug_selftest(None) == -1 and b"not a checked build" in L.disco_last_error()
