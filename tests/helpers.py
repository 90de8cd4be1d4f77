"""Shared helpers for the tests: constructed traces and plain-Python checks."""
import os

import numpy as np

from paper_2502_11417_b200 import synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def constructed(prompt, out, ttft_s, servers=None, devices=None, sprof=None, dprof=None):
    """Arrays for a hand-made trace (dict usable by both the oracle and the library binding)."""
    n = len(prompt)
    return dict(
        prompt_len=np.asarray(prompt, dtype=np.int32), output_len=np.asarray(out, dtype=np.int32),
        server_ttft_s=np.asarray(ttft_s, dtype=np.float32),
        server_profile=np.zeros(n, np.uint8) if sprof is None else np.asarray(sprof, np.uint8),
        device_profile=np.zeros(n, np.uint8) if dprof is None else np.asarray(dprof, np.uint8),
        servers=servers or [synth.server()], devices=devices or [synth.device(500.0, 20.0)])


def oracle_of(tr):
    from oracle import Oracle
    return Oracle(tr["prompt_len"], tr["output_len"], tr["server_ttft_s"], tr["server_profile"],
                  tr["device_profile"], tr["servers"], tr["devices"])
