"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares,
and its host logic (T, sizing, memory accounting, argument validation) is right.  No kernel
is launched here."""
import ctypes as C
import math
import os
import re

import pytest

from oracle import think_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tk():
    from paper_2407_21018_b200 import build
    build.build()
    from paper_2407_21018_b200 import binding
    return binding


def test_exports_every_declared_symbol(tk):
    hdr = open(os.path.join(ROOT, "include", "think.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(thinK_[A-Za-z_0-9]+)\s*\(", hdr))
    assert {"thinK_score_select", "thinK_compact", "thinK_append", "thinK_decode_attn"} <= declared
    for name in declared:
        assert hasattr(tk.lib, name), name
    assert declared == set(tk.EXPORTS), declared ^ set(tk.EXPORTS)


def test_T_matches_definition(tk):
    for D in (64, 128):
        for lam in (0.0, 0.1, 0.25, 0.3, 0.4, 0.5, 0.6, 0.75, 0.9):
            assert tk.thinK_T(lam, D) == orc.kept_channels(lam, D)
    assert tk.thinK_T(1.0, 128) == 0 and tk.thinK_T(-0.1, 128) == 0 and tk.thinK_T(0.999, 64) == 0


def test_status_strings(tk):
    assert tk.lib.thinK_status_string(0) == b"ok"
    assert b"capacity" in tk.lib.thinK_status_string(tk.ERR_CAPACITY)


def test_cache_bytes_and_memory_model(tk):
    # LLaMA-3-8B-shaped: one 8192-token prompt, lambda 0.4, 64 new tokens
    cfg = tk.make_config(1, 32, 32, 8, 128, 8192, 32, 32, 64, 0.4, tk.BF16)
    s = tk.thinK_cache_bytes(cfg, [8192])
    T = 76
    n_tiles = math.ceil((8192 - 32) / 64)
    assert s.k_thin == 32 * 8 * (n_tiles + 2) * 80 * 64 * 2   # bf16 tiles pad T = 76 to 80 rows; 2 spare tiles per head
    assert s.tail_k == 32 * 8 * math.ceil(96 / 64) * 128 * 64 * 2
    assert s.tail_v == 32 * 8 * 96 * 128 * 2
    assert s.idx == 32 * 8 * T
    assert s.scores == 32 * 8 * 128 * 8
    # the paper's accounting, via the oracle's model (Sec. 3.1 / 3.3)
    want = orc.think_cache_elements([8192], 32, 8, 128, keep=T / 128, S_recent=32, new_tokens=64) * 2
    assert s.model_think_bytes == want
    assert s.model_dense_bytes == orc.kv_cache_elements(1, 8192 + 64, 32, 8, 128) * 2


def test_memory_model_reproduces_sec31_example(tk):
    # Sec. 3.1: LLaMA-2-7B, B = 13, S = 2048 -> 13 GB; lambda = 0 keeps everything
    cfg = tk.make_config(13, 32, 32, 32, 128, 2048, 32, 32, 0, 0.0, tk.BF16)
    s = tk.thinK_cache_bytes(cfg, [2048] * 13)
    assert s.model_dense_bytes == 2 * 13 * 2048 * 32 * 32 * 128 * 2
    assert s.model_think_bytes == s.model_dense_bytes
    assert round(s.model_dense_bytes / 2 ** 30) == 13


def test_ragged_sizes(tk):
    lens = [100, 64 + 32, 33]
    cfg = tk.make_config(3, 2, 4, 4, 64, 128, 32, 32, 8, 0.5, tk.F32)
    s = tk.thinK_cache_bytes(cfg, lens)
    tiles = sum(math.ceil((x - 32) / 64) for x in lens)
    assert s.k_thin == 2 * 4 * (tiles + 3 * 1) * 32 * 64 * 4   # one spare tile (cap = 40 tokens) per head and entry


@pytest.mark.parametrize("kw", [
    dict(D=96), dict(N_q=6, N_kv=4), dict(lam=1.0), dict(lam=-0.5), dict(B=0), dict(dtype=7),
    dict(N_q=64, N_kv=4), dict(criterion=9), dict(S_obs=0),
])
def test_invalid_configs_are_rejected(tk, kw):
    base = dict(B=1, L=1, N_q=4, N_kv=4, D=64, S_max=512, S_obs=32, S_recent=32, max_new_tokens=8, lam=0.5,
                dtype=tk.F32)
    base.update(kw)
    cfg = tk.make_config(**base)
    with pytest.raises(tk.ThinKError) as e:
        tk.thinK_cache_bytes(cfg, [512] * max(1, base["B"]))
    assert e.value.status in (tk.ERR_INVALID_ARG, tk.ERR_UNSUPPORTED)


def test_invalid_lengths_are_rejected(tk):
    cfg = tk.make_config(2, 1, 4, 4, 64, 512, 32, 32, 8, 0.5, tk.F32)
    for lens in ([512, 16], [512, 600], [0, 512]):
        with pytest.raises(tk.ThinKError):
            tk.thinK_cache_bytes(cfg, lens)


def test_null_arguments(tk):
    assert tk.lib.thinK_cache_bytes(None, None, None) == tk.ERR_INVALID_ARG
    assert tk.lib.thinK_destroy(None) == tk.ERR_INVALID_ARG
    assert tk.lib.thinK_tail_len(None, 0) == -1
    h = C.c_void_p()
    cfg = tk.make_config(1, 1, 4, 4, 64, 512, 32, 32, 8, 0.5, tk.F32)
    arr = (C.c_int32 * 1)(512)
    sizes = tk.thinK_cache_bytes(cfg, [512])
    assert tk.lib.thinK_create(C.byref(cfg), arr, C.byref(sizes), None, None, None, None, None, None,
                               C.byref(h)) == tk.ERR_INVALID_ARG
    assert tk.lib.thinK_create(C.byref(cfg), arr, None, 256, 256, 256, 256, None, 256, C.byref(h)) == tk.ERR_INVALID_ARG


@pytest.mark.parametrize("short", ["k_thin", "tail_k", "tail_v", "idx", "workspace", "scores"])
def test_create_refuses_buffers_smaller_than_required(tk, short):
    """thinK_create compares the caller's stated buffer sizes with what the configuration needs; the
    check comes before any device access, so fake (aligned, never dereferenced) pointers do here."""
    cfg = tk.make_config(2, 2, 8, 4, 64, 512, 32, 32, 8, 0.5, tk.BF16)
    lens = [512, 300]
    arr = (C.c_int32 * 2)(*lens)
    have = tk.thinK_cache_bytes(cfg, lens)
    setattr(have, short, getattr(have, short) - 1)
    h = C.c_void_p()
    fake = [4096] * 6                                   # k_thin, tail_k, tail_v, idx, scores, workspace
    st = tk.lib.thinK_create(C.byref(cfg), arr, C.byref(have), *fake, C.byref(h))
    assert st == tk.ERR_CAPACITY and not h.value
    if short == "scores":                               # an absent score buffer needs no size
        pass
