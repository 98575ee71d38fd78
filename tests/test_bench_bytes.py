"""The benchmark's algorithmic-byte accounting against totals worked out by hand from the method's
definition (Sec. 3.1 cache shapes, Sec. 3.3 two-part cache): per (b, layer, key head) a decode step must
move S_p*T + (R+t+1)*D key elements and (S+t+1)*D value elements, a prefill S*D keys in and S_p*T + R*D out."""
import dataclasses
import importlib.util
import os

import pytest

from paper_2407_21018_b200 import workloads as wl

_spec = importlib.util.spec_from_file_location("bench", os.path.join(os.path.dirname(__file__), "..", "bench.py"))
bench = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(bench)

T_OF = {"c1": 32, "c2": 76, "c3": 64, "c4": 51, "c5": 64}


def _by_hand_decode(w, T, t):
    e = w.elem_bytes
    tot = 0
    for S in w.seq_lens:
        keys = (S - w.recent) * T + (w.recent + t + 1) * w.D
        values = (S + t + 1) * w.D
        tot += (keys + values) * e * w.L * w.N_kv
    return tot


@pytest.mark.parametrize("name,step,expect_gb", [
    ("c2", 0, 0.857), ("c3", 0, 12.89), ("c5", 0, 12.89), ("c4", 0, None), ("c4", 255, None),
])
def test_decode_bytes_totals(name, step, expect_gb):
    w = wl.get_config(name)
    got = bench.decode_bytes(w, T_OF[name], step)
    hand = _by_hand_decode(w, T_OF[name], step)
    # the benchmark adds the index list and q / out, a fraction of a percent
    assert hand <= got <= hand * 1.005
    if expect_gb is None:          # ragged, seeded lengths in 2048..4096: between the all-shortest and all-longest batch
        lo = dataclasses.replace(w, seq_lens=(2048,) * w.B)
        hi = dataclasses.replace(w, seq_lens=(4096,) * w.B)
        assert bench.decode_bytes(lo, T_OF[name], step) < got < bench.decode_bytes(hi, T_OF[name], step)
    else:
        assert abs(got / 1e9 - expect_gb) / expect_gb < 0.02


@pytest.mark.parametrize("lam,expect_gb", [(0.0, 17.18), (0.25, 15.03), (0.75, 10.74)])
def test_decode_bytes_lambda_sweep_c5(lam, expect_gb):
    w = dataclasses.replace(wl.get_config("c5"), lam=lam)
    T = int((1 - lam) * w.D + 1e-9)
    assert abs(bench.decode_bytes(w, T, 0) / 1e9 - expect_gb) / expect_gb < 0.01


@pytest.mark.parametrize("name,expect_gb", [("c2", 0.865), ("c3", 12.92), ("c4", None), ("c5", 12.90)])
def test_prefill_bytes_totals(name, expect_gb):
    w = wl.get_config(name)
    got = bench.prefill_bytes(w, T_OF[name])
    e = w.elem_bytes
    hand = sum((S * w.D + (S - w.recent) * T_OF[name] + w.recent * w.D) * e for S in w.seq_lens) * w.L * w.N_kv
    assert hand <= got <= hand * 1.03          # + window queries, recent values, index list
    if expect_gb is not None:
        assert abs(got / 1e9 - expect_gb) / expect_gb < 0.02


def test_value_pruning_and_eviction_accounting_are_consistent():
    w = wl.get_config("c2")
    T, Tv = 76, 89
    # pruning the values can only shrink a decode step, by exactly the dropped prefix value channels
    full, thin = bench.decode_bytes(w, T, 0), bench.decode_bytes(w, T, 0, Tv)
    dropped = sum((S - w.recent) * (w.D - Tv) * w.elem_bytes for S in w.seq_lens) * w.L * w.N_kv
    assert abs((full - thin) - dropped) <= w.D * w.L * w.N_kv * w.B
    # behind an eviction method the cache sees the kept tokens only
    ev = wl.evicted(w, 1024)
    assert bench.decode_bytes(ev, T, 0) < full / 7
    assert bench.prefill_bytes_evicted(ev, T) > bench.prefill_bytes(ev, T)
