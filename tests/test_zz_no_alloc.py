"""The allocation-free TTFT sort against the ordinary load path (needs a GPU).

disco_sort_ttft_ticks_noalloc is for callers that must not allocate device memory when they need the sorted
TTFT sample (a serving process whose pool owns the GPU, code between latency-critical launches, a plug-in
without an allocator).  Its working memory is a fixed array inside the library that every call reuses, so
this test calls it twice in a row with different data and lengths -- the second call sees the first call's
leftovers -- and compares each result, bit for bit, with what disco_load_trace + disco_get_group_tables
give for the same values.  Collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest

from paper_2502_11417_b200 import Trace, DiscoError, synth
from paper_2502_11417_b200.api import sort_ttft_ticks_noalloc, NOALLOC_MAX_N

pytestmark = pytest.mark.gpu


def _via_load(ttft):
    n = len(ttft)
    tr = Trace().load_trace(np.full(n, 10, np.int32), np.full(n, 5, np.int32), ttft, None, None,
                            [synth.server()], [synth.device(500.0, 20.0)])
    _, _, srt = tr.group_tables(0)
    tr.close()
    return srt


def test_two_calls_in_a_row_match_the_load_path():
    import torch
    rng = np.random.default_rng(42)
    first = np.clip(np.exp(rng.normal(-0.5, 0.9, size=150_001)), 1e-3, 600.0).astype(np.float32)
    second = np.clip(np.exp(rng.normal(0.3, 1.1, size=4_097)), 1e-3, 2000.0).astype(np.float32)
    # The first call on a device loads the kernels and looks up the working array's address; it belongs to
    # start-up.  From then on the device's free memory, as the driver reports it, must not move across a call: that
    # figure sees a cudaMalloc made by the library itself, which the framework's own allocator statistics would not.
    warm = torch.ones(1000, dtype=torch.float32, device="cuda")
    sort_ttft_ticks_noalloc(warm, torch.empty(1000, dtype=torch.int32, device="cuda"))
    for ttft in (first, second):                       # the second call runs on the first call's leftovers
        x = torch.from_numpy(ttft).cuda()
        out = torch.empty(len(ttft), dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        free_before, held_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        sort_ttft_ticks_noalloc(x, out)
        assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == held_before
        got = out.cpu().numpy()
        want = _via_load(ttft)
        assert got.shape == want.shape and (got == want).all()      # integer work: bit-exact
        assert (np.diff(got) >= 0).all()
        assert (np.sort(np.rint(ttft.astype(np.float64) * 1e6).astype(np.int64)) == got).all()


def test_limits_are_refused_with_a_clear_error():
    import torch
    big = torch.ones(NOALLOC_MAX_N + 1, dtype=torch.float32, device="cuda")
    out = torch.empty(NOALLOC_MAX_N + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(DiscoError) as ei:
        sort_ttft_ticks_noalloc(big, out)
    assert ei.value.code == -1 and "DISCO_NOALLOC_MAX_N" in str(ei.value)
    # the maximum itself is accepted, and so is an empty input
    sort_ttft_ticks_noalloc(big[:NOALLOC_MAX_N], out[:NOALLOC_MAX_N])
    assert (out[:NOALLOC_MAX_N] == 1_000_000).all()
    sort_ttft_ticks_noalloc(big[:0], out[:0])
    bad = torch.tensor([0.5, float("nan"), 1.0], dtype=torch.float32, device="cuda")
    with pytest.raises(DiscoError) as ei:
        sort_ttft_ticks_noalloc(bad, out[:3])
    assert ei.value.code == -1
    # a failed call leaves the shared array usable
    good = torch.tensor([0.5, 0.25, 1.0], dtype=torch.float32, device="cuda")
    sort_ttft_ticks_noalloc(good, out[:3])
    assert out[:3].tolist() == [250000, 500000, 1000000]
