"""CUDA path against the oracle, through the C ABI (needs a GPU)."""
import numpy as np
import pytest

from paper_2502_11417_b200 import synth, Trace, DiscoError
from parity import full_parity, check_stats, check_pairs
from helpers import constructed

pytestmark = pytest.mark.gpu

MIG, PACE = synth.FLAG_MIGRATION, synth.FLAG_PACING
S_MODE, D_MODE = synth.MODE_SERVER_CONSTRAINED, synth.MODE_DEVICE_CONSTRAINED


def test_config0_full():
    full_parity(synth.make_workload(0), tag="config0")


def test_config1_shape_ragged_tiles():
    # several request chunks and policy tiles, none of them full
    w = synth.make_workload(1, n=7013, n_budgets=21)
    full_parity(w, tag="config1-small")


def test_config2_shape_threshold_grid():
    w = synth.make_workload(2, n=5000, n_budgets=9)
    full_parity(w, tag="config2-small")


def test_config3_shape_long_outputs():
    w = synth.make_workload(3, n=1500, n_budgets=5)
    assert w.output_len.max() > 2048
    full_parity(w, tag="config3-small")


def test_config4_shape_six_groups_two_modes():
    w = synth.make_workload(4, n=9000, n_budgets=7)
    gs, _ = full_parity(w, tag="config4-small")
    assert any(s.n_migrations for s in gs)


def test_config5_shape_paper_device_profiles():
    w = synth.make_workload(5, n=8000, n_budgets=6)
    gs, _ = full_parity(w, tag="config5-small")
    assert any(s.n_migrations for s in gs) and any(s.n_device_won for s in gs)


@pytest.mark.parametrize("flags", [0, PACE, MIG, MIG | PACE])
@pytest.mark.parametrize("mode", [S_MODE, D_MODE])
def test_flag_and_mode_matrix(flags, mode):
    pols = [synth.policy(b, mig_threshold=th, t_m_s=tm, flags=flags | mode)
            for b in (0.0, 0.04, 0.3, 1.0) for th in (0.0, 0.01) for tm in (0.0, 0.45, 1.0)]
    for dear in (False, True):
        w = synth.tiny_workload(17 + dear, 700, n_servers=2, n_devices=2, max_prompt=500, max_out=150,
                                device_dearer=dear)
        full_parity(w, pols, tag=f"matrix flags={flags} mode={mode} dear={dear}")


def test_mixed_timeline_classes_in_one_call():
    # policies differing in r_c, t_m and pacing need separate play-outs inside one evaluation
    pols = [synth.policy(0.5, r_c=5.0), synth.policy(0.5, r_c=12.0, t_m_s=0.5), synth.policy(0.7, flags=MIG),
            synth.policy(0.2, r_c=5.0, t_m_s=3.0), synth.policy(0.9, r_c=40.0), synth.policy(1.0, r_c=5.0)]
    w = synth.tiny_workload(5, 900, max_prompt=800, max_out=200)
    full_parity(w, pols, tag="classes")


def test_generation_slower_than_consumption():
    # r_c above the decode rates: the buffer drains, TBTs follow generation, hand-offs are rare
    pols = [synth.policy(b, r_c=rc, t_m_s=0.2, flags=MIG | PACE | S_MODE) for b in (0.5, 1.0) for rc in (25.0, 60.0)]
    w = synth.tiny_workload(9, 600, max_prompt=300, max_out=300)
    full_parity(w, pols, tag="slow-gen")


def test_long_outputs_with_and_without_clamping():
    # mean output above 512 tokens (four requests per warp round); r_c = 5 never clamps, r_c = 30 does for the
    # phone-class device (10 tok/s), so both forms of the clamp-free kernel and its to-do list run
    w = synth.make_workload(3, n=1200, n_budgets=3)
    assert w.output_len.mean() >= 512
    pols = [synth.policy(b, r_c=rc, t_m_s=tm) for b in (0.3, 1.0) for rc, tm in ((5.0, 1.0), (30.0, 0.3), (5.0, 4.0))]
    full_parity(w, pols, tag="long-outputs")


def test_consumption_interval_equal_to_slowest_token():
    # tau = T + J exactly for the device (100,000 + 5,000 ticks): intervals of zero slack, never negative
    w = synth.make_workload(3, n=900, n_budgets=2)
    pols = [synth.policy(b, r_c=1e6 / 105000.0, t_m_s=tm) for b in (0.5, 1.0) for tm in (0.5, 2.0)]
    gs, _ = full_parity(w, pols, tag="tau-equals-slowest")
    tr = Trace.from_workload(w)
    tr.eval_policies(pols, w.seed)
    assert tr.prep(0, 0).tau == 105000
    tr.close()


@pytest.mark.parametrize("top_s", [16.70, 16.80, 1500.0])
def test_sorted_ticks_around_the_fourth_radix_byte(top_s):
    # one-group traces whose largest TTFT lies just below 2^24 ticks (the fourth radix pass skips itself), just
    # above it and far above it: the sorted sample, the knots and everything derived from them
    w = synth.make_workload(1, n=6000, n_budgets=5)
    w.server_ttft_s[::97] *= np.float32(7.0)
    w.server_ttft_s[5] = np.float32(top_s)
    assert float(w.server_ttft_s.max()) == float(np.float32(top_s))
    full_parity(w, [synth.policy(b, flags=MIG | PACE | D_MODE) for b in (0.02, 0.3, 0.8)] + w.policies,
                tag=f"radix-top-{top_s}")


def test_stochastic_baselines_and_expected_length():
    # Stoch-S / Stoch-D routing and the expected-length trigger, mixed with ordinary policies in one call
    STOCH = synth.FLAG_STOCHASTIC
    pols = [synth.policy(b, flags=STOCH | f | md) for b in (0.0, 0.3, 0.77, 1.0) for f in (PACE, MIG | PACE)
            for md in (S_MODE, D_MODE, synth.MODE_AUTO)]
    pols += [synth.policy(b, mig_threshold=th, expected_len=E) for b in (0.4, 1.0) for th in (0.0, 0.02)
             for E in (0, 5, 64, 128, 4096)]
    # random routing takes precedence over the Eq. 1-2 wait rule: one endpoint, no race
    both = [synth.policy(b, flags=STOCH | synth.FLAG_BETA_RULE | MIG | PACE | md, l_immediate=li)
            for b in (0.3, 0.77) for md in (D_MODE, synth.MODE_AUTO) for li in (0, 50)]
    first_both = len(pols)
    pols += both
    for dear in (False, True):
        w = synth.tiny_workload(31 + dear, 3000, n_servers=2, n_devices=2, max_prompt=600, max_out=200,
                                device_dearer=dear)
        gs, _ = full_parity(w, pols, tag=f"next dear={dear}")
        assert gs[0].n_race == 0 and gs[3].n_race == 0
        assert all(gs[first_both + k].n_race == 0 and gs[first_both + k].n_migrations == 0 for k in range(len(both)))
        # a tile of such policies alone (staged histogram increments in the reduction kernel)
        full_parity(w, both, tag=f"stoch+beta dear={dear}")


def test_linear_wait_rule():
    # Eq. 1-2: waits min(beta l, w_tail) with an immediate-start threshold, beside Algorithm 2's policies
    BETA = synth.FLAG_BETA_RULE
    pols = [synth.policy(b, flags=BETA | f | md, l_immediate=li)
            for b in (0.0, 0.03, 0.05, 0.2, 0.5, 0.9, 1.0) for li in (0, 40, 4096)
            for f, md in ((PACE, D_MODE), (MIG | PACE, synth.MODE_AUTO), (MIG, S_MODE))]
    pols += [synth.policy(b, flags=MIG | PACE | D_MODE) for b in (0.2, 0.9)]
    for dear in (False, True):
        w = synth.tiny_workload(41 + dear, 3000, n_servers=2, n_devices=2, max_prompt=600, max_out=200,
                                device_dearer=dear)
        full_parity(w, pols, tag=f"beta dear={dear}")
    # one group at a workload's own length mix, so that the slope search runs over a full length histogram
    w = synth.make_workload(1, n=20000, n_budgets=4)
    full_parity(w, [synth.policy(b, flags=BETA | MIG | PACE | D_MODE, l_immediate=li)
                    for b in (0.1, 0.4, 0.8) for li in (0, 64)], tag="beta workload1")


def test_buffer_search_paths():
    # the hand-off search under clamping (generation sometimes slower than consumption), for shallow
    # buffers, buffers deeper than a warp's delivery-time history, and buffers that never fill
    srv, dev = [synth.server(tbt_s=0.050, jitter=0.3)], [synth.device(900.0, 22.0, jitter=0.3)]
    for dear in (False, True):
        if dear:
            dev = [synth.device(900.0, 22.0, jitter=0.3, c_prefill=5e-3, c_decode=5e-3)]
        rng = np.random.default_rng(77 + dear)
        n = 500
        tr = constructed(rng.integers(1, 600, size=n), rng.integers(1, 1500, size=n),
                         rng.uniform(0.01, 1.5, size=n), servers=srv, devices=dev)
        w = synth.Workload(name="search", seed=11, materialise=True, policies=[], **tr)
        pols = [synth.policy(1.0, r_c=rc, t_m_s=tm, flags=MIG | PACE | md)
                for md in (S_MODE, D_MODE) for rc, tm in ((18.0, 0.3), (18.0, 15.0), (21.0, 14.0), (25.0, 2.0),
                                                          (16.0, 40.0), (30.0, 0.05))]
        gs, _ = full_parity(w, pols, tag=f"search dear={dear}")
        assert any(s.n_migrations for s in gs)


def test_edge_cases():
    # single-token outputs, longest outputs, extreme prompts, ties at S = Td, one request
    tr = constructed([1, 4096, 45, 45, 45, 7, 4096], [1, 8192, 2, 1, 8192, 3, 1],
                     [1e-3, 400.0, 0.1, 0.1, 0.100001, 0.05, 1.0],
                     devices=[synth.device(500.0, 20.0, ttft_intercept_s=0.01, jitter=0.05)],
                     servers=[synth.server(jitter=0.2)])
    w = synth.Workload(name="edges", seed=3, materialise=True, policies=[], **tr)
    pols = [synth.policy(b, flags=f | md) for b in (0.0, 0.5, 1.0) for f in (MIG | PACE, PACE) for md in (S_MODE, D_MODE)]
    full_parity(w, pols, tag="edges")
    # the largest server TTFT the loader accepts, with outputs short enough for the 32-bit tick range
    far = synth.Workload(name="far", seed=2, materialise=True, policies=[],
                         **constructed([300, 20, 4096], [500, 40, 2], [2000.0, 1999.5, 0.2],
                                       devices=[synth.device(500.0, 20.0, c_prefill=5e-3, c_decode=5e-3)]))
    full_parity(far, [synth.policy(b) for b in (0.0, 0.5, 1.0)], tag="far")
    one = synth.Workload(name="one", seed=1, materialise=True, policies=[],
                         **constructed([100], [50], [0.2]))
    full_parity(one, [synth.policy(1.0)], tag="one")


def test_empty_trace_and_reload():
    w = synth.tiny_workload(1, 300)
    t = Trace.from_workload(w)
    e = constructed([], [], [])
    t.load_trace(e["prompt_len"], e["output_len"], e["server_ttft_s"], None, None, e["servers"], e["devices"])
    t.eval_policies([synth.policy(0.5)], 0)
    s = t.reduce_stats()[0]
    assert s.n_requests == 0 and s.total_cost == 0.0 and s.tok_server == 0
    # reload a larger trace into the same context
    w2 = synth.tiny_workload(2, 2000)
    t.load_trace(w2.prompt_len, w2.output_len, w2.server_ttft_s, w2.server_profile, w2.device_profile,
                 w2.servers, w2.devices)
    from oracle import Oracle
    t.eval_policies(w2.policies, 7)
    gs = t.reduce_stats()
    os_, _ = Oracle.from_workload(w2).eval(w2.policies, 7)
    check_stats(gs, os_, t.histograms, "reload")


def test_device_resident_inputs_match_host_inputs():
    import torch
    w = synth.make_workload(4, n=4000, n_budgets=3)
    a = Trace.from_workload(w)
    a.eval_policies(w.policies, 4)
    sa = a.reduce_stats()
    dev = [torch.from_numpy(x).cuda() for x in (w.prompt_len, w.output_len, w.server_ttft_s, w.server_profile,
                                                 w.device_profile)]
    b = Trace().load_trace(*dev, w.servers, w.devices)
    b.eval_policies(w.policies, 4)
    sb = b.reduce_stats()
    for p in range(len(w.policies)):
        assert bytes(sa[p]) == bytes(sb[p])


def test_buffer_test_on_an_exact_tie():
    # jitter-free server at T = tau / 2 with a buffer of three: d_3 = g_5 exactly, so the strict test hands over at 6
    srv = [synth.server(tbt_s=0.050)]
    tr = constructed([100] * 4, [5, 6, 7, 20], [1e-6] * 4, servers=srv, devices=[synth.device(200.0, 10.0)])
    w = synth.Workload(name="tie", seed=2, materialise=True, policies=[], **tr)
    pol = synth.policy(1.0, t_m_s=0.3, r_c=10.0, flags=MIG | PACE | S_MODE)
    gs, _ = full_parity(w, [pol], tag="buffer-tie")
    tr2 = Trace.from_workload(w)
    out = tr2.alloc_pair_outputs(1, fields=["mig_at"])
    tr2.eval_policies([pol], w.seed, out)
    assert out["mig_at"][0].tolist() == [0, 0, 6, 6]
    tr2.close()


def test_selection_prefers_the_tail_over_the_mean():
    # two policies whose order by P99 TTFT is the reverse of their order by mean TTFT
    w = synth.make_workload(1, n=4000, n_budgets=3)
    pols = [synth.policy(0.6, flags=PACE | S_MODE), synth.policy(0.4, flags=PACE | D_MODE)]
    gs, _ = full_parity(w, pols, tag="tail-vs-mean")
    assert gs[0].bin_p99_ttft < gs[1].bin_p99_ttft and gs[0].mean_ttft_s > gs[1].mean_ttft_s
    tr = Trace.from_workload(w)
    tr.eval_policies(pols, w.seed)
    tr.reduce_stats()
    assert tr.select_policy(1e30, 10.0) == (0, 0)
    tr.close()


def test_algorithm1_on_unequal_device_costs_and_exchange_rate():
    # automatic mode: min(lambda c_d) against max(c_s).  Device A: prefill cheap, decode dear -> server-constrained
    # (a max over the device costs would say otherwise); device B: cheap per unit but lambda = 3 -> device-constrained
    devs = [synth.device(500.0, 20.0, c_prefill=0.5e-3, c_decode=3e-3, lam=1.0),
            synth.device(500.0, 20.0, c_prefill=0.4e-3, c_decode=0.4e-3, lam=3.0)]
    w = synth.tiny_workload(8, 1500, n_servers=1, n_devices=2, max_prompt=400, max_out=120)
    w.devices = devs
    pols = [synth.policy(b, flags=MIG | PACE | synth.MODE_AUTO) for b in (0.2, 0.7)]
    full_parity(w, pols, tag="alg1-costs")
    tr = Trace.from_workload(w)
    tr.eval_policies(pols, w.seed)
    assert not tr.prep(0, 0).device_constrained and tr.prep(1, 0).device_constrained
    tr.close()


def test_profile_ids_with_unequal_numbers_of_servers_and_devices():
    # 2 server x 3 device profiles with distinct intervals and device TTFTs (group = server id * 3 + device id)
    srv = [synth.server(tbt_s=0.030, jitter=0.2), synth.server(tbt_s=0.045, jitter=0.1)]
    dev = [synth.device(500.0, 20.0, jitter=0.05), synth.device(250.0, 10.0, jitter=0.05, ttft_intercept_s=0.02),
           synth.device(1000.0, 40.0, jitter=0.1, c_prefill=5e-3, c_decode=5e-3)]
    rng = np.random.default_rng(5)
    n = 2400
    tr = constructed(rng.integers(1, 600, size=n), rng.integers(1, 200, size=n), rng.lognormal(-1.0, 0.8, size=n),
                     servers=srv, devices=dev, sprof=rng.integers(0, 2, size=n), dprof=rng.integers(0, 3, size=n))
    w = synth.Workload(name="2x3", seed=6, materialise=True, policies=[], **tr)
    gs, _ = full_parity(w, [synth.policy(b, mig_threshold=th) for b in (0.1, 0.5, 0.9) for th in (0.0, 0.05)], tag="2x3")
    assert any(s.n_migrations for s in gs)


def test_bins_around_the_end_of_the_linear_region():
    # TTFTs and inter-token intervals of 29 to 34 ticks: bins 0..31 hold one tick each, the octaves start at 32
    srv = [synth.server(tbt_s=31e-6), synth.server(tbt_s=32e-6)]
    ttft = np.array([29e-6, 30e-6, 31e-6, 32e-6, 33e-6, 34e-6] * 2, np.float32)
    tr = constructed([50] * 12, [4] * 12, ttft, servers=srv, sprof=[0] * 6 + [1] * 6)
    w = synth.Workload(name="bins", seed=1, materialise=True, policies=[], **tr)
    gs, _ = full_parity(w, [synth.policy(0.0, flags=D_MODE), synth.policy(0.0, flags=PACE | D_MODE, r_c=1e6 / 31.0)],
                        tag="bins-31-32")
    assert gs[0].n_server_only == 12


def test_budget_equal_to_the_tail_ratio():
    # b = alpha exactly: Algorithm 2 stays in its tail-only branch (every length waits w_tail)
    w = synth.make_workload(1, n=3000, n_budgets=2)
    pols = [synth.policy(b, alpha=a, flags=MIG | PACE | D_MODE) for b, a in ((0.05, 0.05), (0.3, 0.3), (0.30000001, 0.3),
                                                                            (0.31, 0.3))]
    full_parity(w, pols, tag="b-equals-alpha")
    tr = Trace.from_workload(w)
    tr.eval_policies(pols, w.seed)
    assert tr.prep(0, 0).l_star == 0 and tr.prep(0, 1).l_star == 0 and tr.prep(0, 3).l_star > 0
    tr.close()


def test_single_token_outputs_never_hand_over():
    # an output of one token leaves nothing to migrate, whatever the trigger says (expected length 128, no buffer)
    for dear in (False, True):
        w = synth.tiny_workload(23 + dear, 1200, n_servers=2, n_devices=2, max_prompt=300, max_out=30, device_dearer=dear)
        w.output_len[::3] = 1
        pols = [synth.policy(b, flags=f | md, expected_len=E, t_m_s=tm) for b in (0.3, 1.0) for f in (MIG, MIG | PACE)
                for md in (S_MODE, D_MODE) for E in (0, 128) for tm in (0.0, 1.0)]
        gs, _ = full_parity(w, pols, tag=f"single-token dear={dear}")
        assert any(s.n_migrations for s in gs)


def test_seed_above_32_bits():
    w = synth.make_workload(1, n=3000, n_budgets=4)
    full_parity(w, seed=0x123456789ABCDEF0, tag="seed-hi")


def test_handoff_with_one_token_left():
    # jitter-free streams that fill a buffer of five at token 6: outputs of 5 to 9 tokens, so that the hand-off
    # falls on the last token that still leaves one to generate, or no longer fits
    tr = constructed([100] * 5 + [400] * 5, [5, 6, 7, 8, 9] * 2, [1e-6] * 10, devices=[synth.device(200.0, 10.0)])
    w = synth.Workload(name="last-token", seed=3, materialise=True, policies=[], **tr)
    gs, _ = full_parity(w, [synth.policy(1.0, t_m_s=1.0, r_c=5.0, flags=MIG | PACE | S_MODE),
                            synth.policy(1.0, t_m_s=0.0, r_c=5.0, flags=MIG | PACE | S_MODE)], tag="last-token")
    assert gs[0].n_migrations == 6 and gs[1].n_migrations == 10


def test_quantile_rank_reached_at_a_bin_boundary():
    # four requests alone in their TTFT bins: the nearest rank of P50 falls exactly on the end of a bin
    tr = constructed([50, 60, 70, 80], [3, 4, 5, 6], np.array([0.008, 0.001, 0.004, 0.002], dtype=np.float32))
    w = synth.Workload(name="rank", seed=1, materialise=True, policies=[], **tr)
    gs, _ = full_parity(w, [synth.policy(0.0, flags=PACE | D_MODE), synth.policy(1.0, flags=PACE | S_MODE)], tag="rank")
    assert gs[0].n_server_only == 4


def test_pinned_host_inputs_read_in_place_match_pageable_ones():
    # one profile group: page-locked host arrays are read by the ingestion kernel in place, pageable ones are
    # copied first; both must give the same tables and statistics (and the oracle's)
    import torch
    from parity import check_tables
    from oracle import Oracle
    w = synth.make_workload(1, n=30011, n_budgets=7)
    w.server_profile = None; w.device_profile = None          # optional arrays left out
    a = Trace.from_workload(w)
    a.eval_policies(w.policies, 9)
    sa = a.reduce_stats()
    pinned = [torch.from_numpy(x).pin_memory() for x in (w.prompt_len, w.output_len, w.server_ttft_s)]
    b = Trace().load_trace(*pinned, None, None, w.servers, w.devices)
    check_tables(b, Oracle.from_workload(w), "pinned")
    b.eval_policies(w.policies, 9)
    sb = b.reduce_stats()
    for p in range(len(w.policies)):
        assert bytes(sa[p]) == bytes(sb[p])
    pinned[0][17] = 0                                          # validation still sees the in-place arrays
    with pytest.raises(DiscoError):
        Trace().load_trace(*pinned, None, None, w.servers, w.devices)


def test_pinned_host_inputs_of_several_groups_and_staged_copies():
    # six groups: page-locked arrays are read in place as well (packed copies of the lengths feed the partition);
    # arrays_on_device = 2 copies them with the copy engine instead.  All three routes give identical records.
    import torch
    from parity import check_tables
    from oracle import Oracle
    w = synth.make_workload(4, n=25013, n_budgets=3)
    cols = (w.prompt_len, w.output_len, w.server_ttft_s, w.server_profile, w.device_profile)
    a = Trace.from_workload(w)                                  # pageable numpy arrays: copied
    a.eval_policies(w.policies, 9)
    sa = a.reduce_stats()
    pinned = [torch.from_numpy(x).pin_memory() for x in cols]
    for staged in (False, True):
        b = Trace().load_trace(*pinned, w.servers, w.devices, staged_copy=staged)
        check_tables(b, Oracle.from_workload(w), f"pinned staged={staged}")
        b.eval_policies(w.policies, 9)
        sb = b.reduce_stats()
        for p in range(len(w.policies)):
            assert bytes(sa[p]) == bytes(sb[p]), (staged, p)
        b.close()
    pinned[3][11] = 7                                          # validation still sees the in-place arrays
    with pytest.raises(DiscoError):
        Trace().load_trace(*pinned, w.servers, w.devices)


def test_non_default_stream_and_partial_outputs():
    import torch
    w = synth.make_workload(1, n=3000, n_budgets=4)
    st = torch.cuda.Stream()
    t = Trace.from_workload(w, stream=st)
    out = t.alloc_pair_outputs(4, ["ttft_s", "decision"])
    with torch.cuda.stream(st):
        t.eval_policies(w.policies, 1, out)
        gs = t.reduce_stats()
    from oracle import Oracle
    os_, oout = Oracle.from_workload(w).eval(w.policies, 1, pairs=True)
    check_stats(gs, os_, t.histograms, "stream")
    assert (out["decision"].cpu().numpy() == oout["decision"]).all()


def test_invalid_inputs_are_rejected():
    ok = constructed([10, 20], [5, 5], [0.3, 0.4])
    def load(**kw):
        d = dict(ok); d.update(kw)
        return Trace().load_trace(d["prompt_len"], d["output_len"], d["server_ttft_s"], d["server_profile"],
                                  d["device_profile"], d["servers"], d["devices"])
    for bad in [dict(prompt_len=np.array([0, 5], np.int32)), dict(prompt_len=np.array([4097, 5], np.int32)),
                dict(output_len=np.array([5, 8193], np.int32)), dict(output_len=np.array([0, 1], np.int32)),
                dict(server_ttft_s=np.array([np.nan, 1.0], np.float32)),
                dict(server_ttft_s=np.array([0.0, 1.0], np.float32)),
                dict(server_ttft_s=np.array([np.inf, 1.0], np.float32)),
                dict(server_profile=np.array([0, 1], np.uint8)),
                dict(servers=[synth.server(tbt_s=0.0)]), dict(devices=[synth.device(0.0, 20.0)]),
                dict(servers=[synth.server(jitter=1.5)])]:
        with pytest.raises(DiscoError) as ei:
            load(**bad)
        assert ei.value.code == -1
    t = load()
    for badpol in [synth.policy(1.5), synth.policy(0.5, alpha=0.0), synth.policy(0.5, mig_threshold=-1.0),
                   synth.policy(0.5, r_c=0.0), synth.policy(0.5, flags=3 << 2), synth.policy(0.5, flags=1 << 6),
                       synth.policy(0.5, flags=synth.FLAG_BETA_RULE, l_immediate=4097),
                   synth.policy(float("nan"))]:
        with pytest.raises(DiscoError) as ei:
            t.eval_policies([badpol], 0)
        assert ei.value.code == -1
    with pytest.raises(DiscoError):
        t.reduce_stats()                      # nothing evaluated
    # a stream that could outlast the 32-bit tick range is refused, not wrapped
    slow = constructed([10], [8192], [0.3])
    t2 = Trace().load_trace(slow["prompt_len"], slow["output_len"], slow["server_ttft_s"], None, None,
                            slow["servers"], slow["devices"])
    with pytest.raises(DiscoError) as ei:
        t2.eval_policies([synth.policy(0.5, r_c=2.0)], 0)
    assert ei.value.code == -1


def _work(w, pols):
    tr = Trace.from_workload(w)
    tr.eval_policies(pols, w.seed)
    tr.reduce_stats()
    counts = tr.work_counts()
    tr.close()
    return counts


def test_zone_by_zone_reduction_and_what_it_leaves_to_the_pair_kernel():
    # ascending budgets: a tile's policies are ordered, so requests are settled against runs of policies; what the
    # runs cannot express goes pair by pair.  Every variant must give the oracle's numbers.
    for dear in (False, True):                     # Algorithm 3 tiles, Algorithm 2 tiles
        w = synth.tiny_workload(51 + dear, 6000, n_servers=2, n_devices=1, max_prompt=900, max_out=160, device_dearer=dear)
        grid = synth.budget_grid(40)
        # one overhead per tile: nothing but the odd request is left over
        plain = [synth.policy(b, mig_threshold=0.004) for b in grid]
        full_parity(w, plain, tag=f"zones plain dear={dear}")
        zone, left, _, corr = _work(w, plain)
        assert zone > 0.9 * w.n * len(plain) and corr > 0
        # overheads that alternate inside a tile: requests whose saving lies between them are left to the pair kernel
        mixed = [synth.policy(b, mig_threshold=(0.0, 0.05, synth.INF)[k % 3]) for k, b in enumerate(grid)]
        full_parity(w, mixed, tag=f"zones mixed overheads dear={dear}")
        zone, left, _, _ = _work(w, mixed)
        assert zone > 0 and left > 0
        # many budgets at or below the tail ratio (each its own w_tail), and budgets that repeat (equal thresholds)
        low = [synth.policy(b, alpha=0.3) for b in sorted(list(synth.budget_grid(24)) + [0.1, 0.1, 0.5, 0.5, 0.5])]
        full_parity(w, low, tag=f"zones low budgets dear={dear}")
        # the caller's order does not matter: the library lines like policies up by budget itself
        rng = np.random.default_rng(7)
        shuffled = [plain[k] for k in rng.permutation(len(plain))]
        full_parity(w, shuffled, tag=f"zones shuffled dear={dear}")
        assert _work(w, shuffled)[0] > 0.9 * w.n * len(plain)
        # random routing has no ordered thresholds: such tiles go pair by pair
        stoch = [synth.policy(b, flags=synth.FLAG_STOCHASTIC | PACE) for b in grid]
        full_parity(w, stoch, tag=f"zones none dear={dear}")
        assert _work(w, stoch)[0] == 0
        # pacing off: no zone kernel at all
        nopace = [synth.policy(b, flags=MIG) for b in grid]
        full_parity(w, nopace, tag=f"zones pacing off dear={dear}")
        assert _work(w, nopace)[0] == 0


def test_more_than_32_policy_tiles_use_several_flag_words():
    # 1100 policies = 35 tiles: two flag words per request; overheads alternate so that requests are flagged in
    # tiles of both words
    w = synth.tiny_workload(61, 1500, n_servers=1, n_devices=2, max_prompt=700, max_out=120, device_dearer=True)
    pols = [synth.policy(b, mig_threshold=(0.0, 0.03)[k % 2]) for k, b in enumerate(synth.budget_grid(1100))]
    full_parity(w, pols, select=False, tag="35 tiles")
    zone, left, _, _ = _work(w, pols)
    assert zone > 0 and left > 0


def test_one_prompt_length_and_lengths_at_the_ends():
    # every request in one bucket of the internal order: a chunk is one segment (or a threshold's own), and all
    # lanes of a warp meet in one row and one histogram bin
    grid = synth.budget_grid(70)                   # three policy tiles: a family of several tiles
    for dear in (False, True):
        w = synth.tiny_workload(71 + dear, 5000, n_servers=1, n_devices=1, max_prompt=900, max_out=120, device_dearer=dear)
        w.prompt_len[:] = 300
        full_parity(w, [synth.policy(b, mig_threshold=0.004) for b in grid], tag=f"one length dear={dear}")
        # only the shortest and the longest prompt there is
        w.prompt_len[:] = np.where(np.arange(w.n) % 3 == 0, 1, 4096).astype(np.int32)
        full_parity(w, [synth.policy(b, mig_threshold=0.004) for b in grid], tag=f"lengths 1 and 4096 dear={dear}")


def test_more_groups_than_fit_the_scatter_in_shared_memory():
    # 3 x 3 = 9 groups: the internal request order is built with one add per warp and bucket to the global cursors
    # (the length histograms of more than six groups do not fit the slice-wise kernel's shared memory)
    w = synth.tiny_workload(73, 9000, n_servers=3, n_devices=3, max_prompt=600, max_out=100)
    full_parity(w, [synth.policy(b, mig_threshold=0.01) for b in synth.budget_grid(40)], tag="nine groups")
    zone, left, _, _ = _work(w, [synth.policy(b, mig_threshold=0.01) for b in synth.budget_grid(40)])
    assert zone + left == w.n * 40


def test_family_whose_first_tile_alone_has_longer_waits():
    # Algorithm 2 along 128 ascending budgets: the lowest budgets wait longest (w_tail falls until it settles), so a
    # family of four tiles stays whole and requests under which the device wins after such a wait are left to the
    # pair kernel for the first tile only
    w = synth.tiny_workload(74, 20000, n_servers=1, n_devices=1, max_prompt=2000, max_out=200, device_dearer=True)
    pols = [synth.policy(b, mig_threshold=th) for th in (0.0, synth.INF) for b in synth.budget_grid(128)]
    full_parity(w, pols, select=False, tag="four-tile families with waits")
    zone, left, settled, _ = _work(w, pols)
    assert zone + left == w.n * len(pols)
    assert left < 0.1 * zone
    assert settled <= 2 * w.n                      # one sweep per request and family, not per tile
