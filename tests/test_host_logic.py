"""CPU-only checks of the CUDA library's host side: exported symbols and Algorithm 3's
bookkeeping (compared with the oracle's call log)."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2502_07861_b200 as bk
from oracle import OracleParams, OracleStream

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "balancekv.h")).read()
    declared = sorted(set(re.findall(r"\b(balancekv_[a-z_0-9]+)\s*\(", header)))
    assert "balancekv_stream_append" in declared and "balancekv_compress" in declared
    assert "balancekv_decode_attn" in declared
    lib = ctypes.CDLL(bk.load()._name)
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(set(bk.EXPORTS)) == [d for d in declared]


def test_strerror_and_argument_errors_without_a_device():
    lib = bk.load()
    assert lib.balancekv_strerror(0) == b"ok"
    assert b"invalid" in lib.balancekv_strerror(-1)
    assert lib.balancekv_create(None, None) == bk.binding.E_INVAL
    cfg = bk.Config(1, 1, 1, 1, 100, 1, 256, 1, 1024, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0)   # head_dim 100
    h = ctypes.c_void_p()
    assert lib.balancekv_create(ctypes.byref(cfg), ctypes.byref(h)) == bk.binding.E_INVAL
    assert lib.balancekv_plan_calls(3, 1, 0, None, 0, None, 0) == bk.binding.E_INVAL


@pytest.mark.parametrize("t,T,W,chunks", [
    (8, 1, 0, [64]), (8, 3, 0, [8 * 13]), (16, 2, 0, [50, 40, 91]), (16, 4, 0, [16] * 20),
    (16, 3, 24, [100, 3, 97]), (8, 2, 40, [20, 20, 20, 1, 1, 1, 100]), (4, 3, 0, [1] * 70), (64, 2, 5, [1000, 7, 640]),
])
def test_schedule_matches_oracle_call_log(t, T, W, chunks):
    d = 4
    rng = np.random.default_rng(0)
    o = OracleStream(OracleParams(d=d, t=t, T=T, W=W, max_tokens=1 << 20))
    want = []
    seen = 0
    total = 0
    for e, n in enumerate(chunks):
        o.append(rng.standard_normal((n, d)), rng.standard_normal((n, d)))
        o.compress()
        calls = o.calls()
        want += [(e, c["level"], c["ordinal"]) for c in calls[seen:]]
        seen = len(calls)
        total += n
    got = bk.plan_calls(t, T, W, np.cumsum(chunks))
    assert got == want


def test_schedule_T0_runs_nothing():
    assert bk.plan_calls(8, 0, 0, [100, 200]) == []


def test_reference_arm_of_the_bench_prints_the_contract_line():
    """`bench.py --impl reference` times the oracle on the host cores and prints one JSON line with
    the keys the measurement contract asks for (no GPU involved)."""
    import json
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=300, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "impl", "cpu_baseline", "e2e", "gpu_launches"):
        assert key in line, key
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0 and line["vs_baseline"] is None
