"""Seeded synthetic traces, endpoint profiles and policy grids.

This module only draws inputs.  It holds none of the method's arithmetic
(no tick conversion, no hashing, no policy rule), so the CUDA library and the
CPU oracle can both be fed from it without sharing any logic.

The five workloads are synthetic stand-ins for the paper's request traces
(Sec. 5.1: Alpaca prompts against four commercial services, three phone
profiles), which are not redistributable.  Their shapes follow the paper's own
scalability experiment (Sec. 5.2), which fits log-normal prompt lengths and
server TTFTs to its real trace.

Draw order per workload, all from ``numpy.random.Generator(PCG64(seed))``:
prompt lengths, output lengths, TTFT base normals, mixture uniforms, mixture
values, server-profile ids, device-profile ids.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

FLAG_MIGRATION = 1
FLAG_PACING = 2
MODE_AUTO = 0 << 2
MODE_DEVICE_CONSTRAINED = 1 << 2
MODE_SERVER_CONSTRAINED = 2 << 2
FLAG_BETA_RULE = 32         # device-constrained phase 2 as in the body text: w(l) = min(beta l, w_tail)
FLAG_STOCHASTIC = 16        # Stoch-S / Stoch-D baseline: random routing to the constrained endpoint with probability b

INF = float("inf")


@dataclass
class Workload:
    name: str
    prompt_len: np.ndarray      # int32 [n]
    output_len: np.ndarray      # int32 [n]
    server_ttft_s: np.ndarray   # float32 [n]
    server_profile: np.ndarray  # uint8 [n]
    device_profile: np.ndarray  # uint8 [n]
    servers: List[Dict[str, float]]
    devices: List[Dict[str, float]]
    policies: List[Dict[str, float]]
    seed: int                   # seed of the per-token jitter hash
    materialise: bool           # per-pair outputs written out?
    select: Dict[str, float] = field(default_factory=dict)

    @property
    def n(self) -> int:
        return int(self.prompt_len.shape[0])

    @property
    def n_policies(self) -> int:
        return len(self.policies)


def _lengths(rng, n, mu, sigma, lo, hi):
    x = np.exp(rng.normal(mu, sigma, size=n))
    return np.clip(np.rint(x), lo, hi).astype(np.int32)


def server(tbt_s=0.030, jitter=0.0, c_prefill=1.0e-3, c_decode=1.0e-3):
    return dict(tbt_s=tbt_s, jitter=jitter, c_prefill=c_prefill, c_decode=c_decode)


def device(prefill_tps, decode_tps, jitter=0.0, c_prefill=0.2e-3, c_decode=0.2e-3,
           lam=1.0, ttft_intercept_s=0.0):
    return dict(prefill_tps=prefill_tps, ttft_intercept_s=ttft_intercept_s,
                decode_tps=decode_tps, jitter=jitter, c_prefill=c_prefill,
                c_decode=c_decode, lam=lam)


def policy(budget, alpha=0.05, mig_threshold=0.0, t_m_s=1.0, r_c=5.0,
           flags=FLAG_MIGRATION | FLAG_PACING | MODE_AUTO, expected_len=0, l_immediate=0):
    return dict(budget=float(np.float32(budget)), alpha=alpha,
                mig_threshold=mig_threshold, t_m_s=t_m_s, r_c=r_c, flags=int(flags), expected_len=int(expected_len),
                l_immediate=int(l_immediate))


def budget_grid(k: int) -> List[float]:
    """k budgets evenly spaced over [0, 1] (a single budget gives 0.5)."""
    if k == 1:
        return [0.5]
    return [float(np.float32(i) / np.float32(k - 1)) for i in range(k)]


_SIZES = {0: 1_000, 1: 100_000, 2: 1_000_000, 3: 4_000_000, 4: 16_000_000, 5: 600_000}


def make_workload(cfg: int, n: Optional[int] = None, n_budgets: Optional[int] = None,
                  replica: int = 0) -> Workload:
    """Build workload ``cfg`` (0..4).  ``n`` / ``n_budgets`` shrink the request
    count / the budget axis for parity tests; distributions stay the same.
    ``replica`` > 0 draws an independent trace of the same shape (one per GPU
    in a multi-GPU run)."""
    if cfg not in _SIZES:
        raise ValueError("cfg must be 0..5")
    n = _SIZES[cfg] if n is None else int(n)
    rng = np.random.Generator(np.random.PCG64(cfg if replica == 0 else [cfg, replica]))

    if cfg == 5:
        return _paper_profiles_workload(rng, n, n_budgets)
    prompt = _lengths(rng, n, 5.5, 1.0, 16, 4096)
    if cfg == 3:
        out = _lengths(rng, n, 6.5, 0.7, 64, 8192)
    else:
        out = _lengths(rng, n, 5.0, 0.8, 8, 2048)
    z = rng.normal(0.0, 1.0, size=n)
    u = rng.random(size=n)

    jit_s, jit_d = (0.0, 0.0) if cfg == 0 else (0.20, 0.05)
    sprof = np.zeros(n, dtype=np.uint8)
    dprof = np.zeros(n, dtype=np.uint8)

    if cfg in (0, 1, 3):
        ttft = np.exp(-1.0 + 0.6 * z)
        mixv = rng.random(size=n)            # drawn to keep the order fixed; unused
        ttft = np.where(u < 0.05, ttft * 4.0, ttft)
        servers = [server(jitter=jit_s)]
        if cfg == 3:
            devices = [device(200.0, 10.0, jitter=jit_d)]
        else:
            devices = [device(500.0, 20.0, jitter=jit_d)]
    elif cfg == 2:
        ttft = np.exp(-0.5 + 0.9 * z)
        mixv = rng.uniform(5.0, 15.0, size=n)
        ttft = np.where(u < 0.02, mixv, ttft)
        servers = [server(jitter=jit_s)]
        devices = [device(1500.0, 40.0, jitter=jit_d)]
    else:
        mixv = rng.uniform(5.0, 15.0, size=n)
        sprof = rng.integers(0, 3, size=n).astype(np.uint8)
        dprof = rng.integers(0, 2, size=n).astype(np.uint8)
        mu = np.array([-1.6, -0.5, 0.3])[sprof]
        sg = np.array([0.3, 0.9, 1.1])[sprof]
        ttft = np.exp(mu + sg * z)
        ttft = np.where((sprof == 1) & (u < 0.02), mixv, ttft)
        servers = [server(jitter=jit_s) for _ in range(3)]
        devices = [device(1500.0, 40.0, jitter=jit_d),
                   device(200.0, 10.0, jitter=jit_d, c_prefill=5.0e-3, c_decode=5.0e-3)]
    ttft = np.clip(ttft, 1e-3, 600.0).astype(np.float32)

    nb_default = {0: 1, 1: 64, 2: 256, 3: 16, 4: 128}[cfg]
    nb = nb_default if n_budgets is None else int(n_budgets)
    thetas = {0: [0.0], 1: [0.0], 2: [0.0, 0.05, 0.2, INF], 3: [0.0],
              4: [0.0, 0.02, 0.05, 0.1, 0.2, 0.4, 0.8, INF]}[cfg]
    policies = [policy(b, mig_threshold=th) for th in thetas for b in budget_grid(nb)]

    select = dict(cost_cap_factor=1.25, tbt_slo_s=0.25)
    return Workload(name=f"config{cfg}", prompt_len=prompt, output_len=out,
                    server_ttft_s=ttft, server_profile=sprof, device_profile=dprof,
                    servers=servers, devices=devices, policies=policies, seed=cfg,
                    materialise=cfg in (0, 1), select=select)


def _paper_profiles_workload(rng, n, n_budgets) -> Workload:
    """Workload 5: the paper's own endpoint constants on a synthetic trace.  Devices: the three phone
    profiles of Sec. 5.1 (prefill/decode tokens/s 31.32/13.93, 51.80/20.14, 79.90/21.47), device cost per
    token = the model's GFLOPs per token (Table 6: prefill at L=64, decode) priced at two exchange rates so
    that Algorithm 1 yields a server-constrained and a device-constrained variant of each (the paper's
    0.3 vs 5 energy_to_money settings, Appendix E); server prices of GPT-4o-mini (Table 8, $ per token);
    outputs capped at the paper's generation limit 128; short instruction-style prompts.  The server TTFT
    column is synthetic (the commercial traces are not available)."""
    prompt = _lengths(rng, n, 3.3, 0.8, 4, 512)
    out = _lengths(rng, n, 5.0, 0.8, 8, 128)
    z = rng.normal(0.0, 1.0, size=n)
    u = rng.random(size=n)
    mixv = rng.uniform(5.0, 15.0, size=n)
    ttft = np.where(u < 0.02, mixv, np.exp(-0.5 + 0.9 * z))
    sprof = np.zeros(n, dtype=np.uint8)
    dprof = rng.integers(0, 6, size=n).astype(np.uint8)
    ttft = np.clip(ttft, 1e-3, 600.0).astype(np.float32)
    servers = [server(jitter=0.20, c_prefill=0.15e-6, c_decode=0.60e-6)]
    phones = [(31.32, 13.93, 0.93, 0.82), (51.80, 20.14, 0.50, 0.42), (79.90, 21.47, 0.45, 0.37)]
    devices = [device(pf, dc, jitter=0.05, c_prefill=cp, c_decode=cd, lam=lam)
               for lam in (0.3e-6, 5.0e-6) for pf, dc, cp, cd in phones]
    nb = 32 if n_budgets is None else int(n_budgets)
    policies = [policy(b, mig_threshold=th, expected_len=128) for th in (0.0, INF) for b in budget_grid(nb)]
    return Workload(name="config5", prompt_len=prompt, output_len=out, server_ttft_s=ttft, server_profile=sprof,
                    device_profile=dprof, servers=servers, devices=devices, policies=policies, seed=5,
                    materialise=False, select=dict(cost_cap_factor=1.25, tbt_slo_s=0.25))


def tiny_workload(seed: int, n: int, *, n_servers=1, n_devices=1, max_prompt=64, max_out=40,
                  policies: Optional[List[Dict[str, float]]] = None, jitter=(0.2, 0.05),
                  device_dearer=False) -> Workload:
    """Small random workload for brute-force and edge-case tests."""
    rng = np.random.Generator(np.random.PCG64(seed))
    prompt = rng.integers(1, max_prompt + 1, size=n).astype(np.int32)
    out = rng.integers(1, max_out + 1, size=n).astype(np.int32)
    ttft = np.clip(np.exp(rng.normal(-1.0, 0.8, size=n)), 1e-3, 600.0).astype(np.float32)
    sprof = rng.integers(0, n_servers, size=n).astype(np.uint8)
    dprof = rng.integers(0, n_devices, size=n).astype(np.uint8)
    servers = [server(tbt_s=0.030 + 0.01 * k, jitter=jitter[0]) for k in range(n_servers)]
    cd = 5.0e-3 if device_dearer else 0.2e-3
    devices = [device(500.0 / (k + 1), 20.0 / (k + 1), jitter=jitter[1], c_prefill=cd, c_decode=cd,
                      ttft_intercept_s=0.01 * k) for k in range(n_devices)]
    if policies is None:
        policies = [policy(b) for b in budget_grid(5)]
    return Workload(name=f"tiny{seed}", prompt_len=prompt, output_len=out, server_ttft_s=ttft,
                    server_profile=sprof, device_profile=dprof, servers=servers, devices=devices,
                    policies=policies, seed=seed, materialise=True,
                    select=dict(cost_cap_factor=1.25, tbt_slo_s=0.25))
