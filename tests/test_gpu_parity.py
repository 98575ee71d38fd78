"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Selected indices and cache contents bit-exact; attention within
1e-2 (bf16 I/O) / 1e-5 (fp32 I/O) max-abs."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import think_oracle as orc
from paper_2407_21018_b200 import workloads as wl

from _harness import (NEAR_TIE_REL, NEAR_TIE_V_REL, assert_attn_close, check_head_selection, compare_cache,
                      compare_selection, make_cache, make_oracle, record_parity, run_case, to64)

pytestmark = pytest.mark.gpu


def test_c1_full():
    """Config 1 exactly as stated: fp32, 4 MHA heads, D=64, S=512, 8 decode steps."""
    r = run_case(wl.get_config("c1"))
    assert r["max_abs"] <= 1e-5


@pytest.mark.parametrize("name,S,L,B,steps", [
    ("c2", 2048 + 37, 2, 1, 6),      # GQA 4:1, RoPE, ragged last tile
    ("c3", 1500, 2, 2, 4),           # batch of equal lengths
    ("c4", 700, 1, 5, 5),            # MHA, ragged batch, outlier channels, T = 51
    ("c5", 3000, 1, 1, 70),          # S_obs = 64; tail grows past one 64-token tile
])
def test_shrunk_configs(name, S, L, B, steps):
    w = wl.shrink(wl.get_config(name), S=S, L=L, B=B, steps=steps)
    run_case(w)


@pytest.mark.parametrize("name,S,L,B,steps", [
    ("c2", 2048 + 37, 3, 1, 2),
    ("c3", 1500, 2, 2, 2),
    ("c4", 700, 2, 5, 2),            # ragged, T = 51 (trailing group of 8 channels)
    ("c5", 9000, 1, 1, 2),
    ("c1", 300, 1, 1, 2),            # fp32
])
def test_prefill_in_one_call(name, S, L, B, steps):
    """thinK_prefill (score + select + compact in one call; for bf16 the one-pass kernel) against the oracle."""
    w = wl.shrink(wl.get_config(name), S=S, L=L, B=B, steps=steps)
    run_case(w, fused=True)


@pytest.mark.parametrize("R,criterion", [(0, 0), (1, 0), (32, 1), (32, 2)])
def test_prefill_in_one_call_variants(R, criterion):
    w = dataclasses.replace(wl.shrink(wl.get_config("c2"), S=1100, L=2, steps=2), S_recent=R)
    run_case(w, fused=True, criterion=criterion)


def test_prefill_in_one_call_equals_two_calls_and_repeats():
    """Same idx and the same key-cache bytes as score_select + compact; a second call on the same
    handle gives the same bytes again."""
    w = wl.shrink(wl.get_config("c4"), S=1300, L=2, B=3, steps=1)
    data = wl.make_prefill(w, device="cuda")
    a, b = make_cache(w, 1), make_cache(w, 1)
    a.score_select(data["Q_obs"], data["K"])
    a.compact(data["K"], data["V"])
    for _ in range(2):
        b.k_thin.zero_()
        b.prefill(data["Q_obs"], data["K"], data["V"])
        torch.cuda.synchronize()
        assert b.device_error() == 0
        assert torch.equal(a.idx_tensor(), b.idx_tensor())
        assert torch.equal(a.k_thin, b.k_thin)
    # per-layer calls
    c = make_cache(w, 1)
    for l in (1, 0):
        c.prefill(data["Q_obs"], data["K"], data["V"], layer0=l, nlayers=1)
    torch.cuda.synchronize()
    assert torch.equal(a.idx_tensor(), c.idx_tensor()) and torch.equal(a.k_thin, c.k_thin)


@pytest.mark.parametrize("name,S,R,keep,every", [
    ("c2", 1000, 32, 32, 40),      # GQA: blocks move at steps 40 and 80 ... while 32 stay unpruned
    ("c4", 500, 100, 0, 30),       # MHA ragged, T = 51: the recent prompt rows move at once
    ("c5", 700, 64, 16, 64),
])
def test_tail_reprune(name, S, R, keep, every):
    """thinK_reprune_tail during decode: cache contents bit-exact and attention within tolerance
    against the oracle that moves the same blocks."""
    w = dataclasses.replace(wl.shrink(wl.get_config(name), S=S, L=2, B=2, steps=100), S_recent=R)
    data = wl.make_prefill(w, device="cpu")
    K, V, Q = data["K"].cuda(), data["V"].cuda(), data["Q_obs"].cuda()
    cache = make_cache(w, w.steps)
    cache.prefill(Q, K, V)
    o = make_oracle(w)
    o.score_select(to64(data["Q_obs"]), to64(data["K"]))
    compare_selection(cache.idx_tensor().cpu().numpy(), None, o, w.name)
    o.compact(to64(data["K"]), to64(data["V"]))
    moved_any = False
    for t in range(w.steps):
        st = wl.make_step(w, t, device="cpu")
        cache.append(st["k_new"].cuda(), st["v_new"].cuda())
        o.append(to64(st["k_new"]), to64(st["v_new"]))
        if t % every == 0:
            before = cache.repruned_len()
            cache.reprune_tail(keep)
            o.reprune(keep)
            moved_any |= cache.repruned_len() > before
            assert cache.tail_len() - cache.repruned_len() == o.K_full[0][0][0].shape[0]
            compare_cache(cache, o, where=f"{w.name} after reprune at step {t}")
        if t % 7 == 0 or t % every <= 1:
            out = cache.decode_attn(st["q"].cuda())
            torch.cuda.synchronize()
            assert_attn_close(to64(out), o.decode_attn(to64(st["q"])), w.dtype, f"{w.name} step {t}")
    assert moved_any
    assert cache.device_error() == 0


def test_tail_reprune_rejects_fp32():
    from paper_2407_21018_b200 import binding as tk
    w = wl.shrink(wl.get_config("c1"), S=200, steps=2)
    data = wl.make_prefill(w, device="cuda")
    c = make_cache(w, 2)
    c.prefill(data["Q_obs"], data["K"], data["V"])
    with pytest.raises(tk.ThinKError) as e:
        c.reprune_tail(0)
    assert e.value.status == tk.ERR_UNSUPPORTED


@pytest.mark.parametrize("name,S,kv,R", [
    ("c2", 1500, 256, 32),                     # GQA bf16, the paper's KV-size range (128..2048)
    ("c2", 900, 128, 0),                       # no recent window: everything thinned
    ("c4", 700, (130, 257, 64), 32),           # MHA, ragged prompts and ragged kept counts, T = 51
    ("c1", 300, 100, 32),                      # fp32 kernels
])
def test_prefill_behind_token_eviction(name, S, kv, R):
    """thinK_prefill_evicted with a per-head list of kept tokens equals the oracle run on the tensors
    an eviction method would hand over (each head's kept rows gathered)."""
    base = wl.get_config(name)
    B = len(kv) if isinstance(kv, tuple) else min(base.B, 2)
    src = dataclasses.replace(wl.shrink(base, S=S, L=min(base.L, 2), B=B, steps=4), S_recent=R)
    data = wl.make_prefill(src, device="cpu")
    tok = wl.make_eviction(src, kv)
    w = wl.evicted(src, kv)
    cache = make_cache(w, w.steps)
    cache.prefill_evicted(data["Q_obs"].cuda(), data["K"].cuda(), data["V"].cuda(), tok.cuda())
    torch.cuda.synchronize()
    assert cache.device_error() == 0
    o = make_oracle(w)
    tok64 = tok.numpy().astype(np.int64)
    Kg = orc.gather_kept(to64(data["K"]), tok64, list(w.seq_lens))
    Vg = orc.gather_kept(to64(data["V"]), tok64, list(w.seq_lens))
    o.score_select(to64(data["Q_obs"]), Kg)
    compare_selection(cache.idx_tensor().cpu().numpy(), cache.scores_tensor().cpu().numpy(), o, w.name)
    o.compact(Kg, Vg)
    compare_cache(cache, o, where=w.name)
    for t in range(w.steps):
        st = wl.make_step(w, t, device="cpu")
        cache.append(st["k_new"].cuda(), st["v_new"].cuda())
        out = cache.decode_attn(st["q"].cuda())
        torch.cuda.synchronize()
        o.append(to64(st["k_new"]), to64(st["v_new"]))
        assert_attn_close(to64(out), o.decode_attn(to64(st["q"])), w.dtype, f"{w.name} step {t}")
    assert cache.device_error() == 0


def test_eviction_list_out_of_range_is_flagged():
    """A kept-token entry outside the source rows is never dereferenced: it is read as row 0 and the
    device error word is set."""
    src = wl.shrink(wl.get_config("c2"), S=400, L=1, steps=1)
    data = wl.make_prefill(src, device="cuda")
    tok = wl.make_eviction(src, 128)
    tok[0, 0, 3, 5] = 400                      # one past the last source row
    w = wl.evicted(src, 128)
    cache = make_cache(w, 1)
    cache.prefill_evicted(data["Q_obs"], data["K"], data["V"], tok.cuda())
    torch.cuda.synchronize()
    assert cache.device_error() != 0


def test_eviction_rejects_bad_arguments():
    from paper_2407_21018_b200 import binding as tk
    src = wl.shrink(wl.get_config("c2"), S=400, L=1, steps=1)
    data = wl.make_prefill(src, device="cuda")
    w = wl.evicted(src, 128)
    cache = make_cache(w, 1)
    short = wl.make_eviction(src, 128)[..., :100].contiguous().cuda()     # list shorter than the kept count
    with pytest.raises(tk.ThinKError) as e:
        cache.prefill_evicted(data["Q_obs"], data["K"], data["V"], short)
    assert e.value.status == tk.ERR_INVALID_ARG
    tok = wl.make_eviction(src, 128).cuda()
    with pytest.raises(tk.ThinKError) as e:                                # source with fewer rows than kept
        cache.prefill_evicted(data["Q_obs"], data["K"][:, :100], data["V"][:, :100], tok)
    assert e.value.status == tk.ERR_INVALID_ARG


@pytest.mark.parametrize("name,S,L,B,lam_v,R,kernel", [
    ("c2", 1100, 2, 1, 0.3, 32, "tcgen05"),    # GQA 4:1 -> 128 window rows per key head, T_v = 89 (rows padded to 96)
    ("c2", 1100, 2, 1, 0.3, 32, "mma_sync"),   # the same through the mma.sync score kernel
    ("c4", 600, 1, 3, 0.5, 32, "tcgen05"),     # MHA -> 32 rows (always mma.sync), ragged batch, T_v = 64
    ("c5", 2100, 1, 1, 0.25, 0, "tcgen05"),    # S_obs = 64 -> 256 rows = two row blocks; no recent window
    ("c5", 2100, 1, 1, 0.25, 0, "mma_sync"),
    ("c2", 700, 1, 2, 0.9, 32, "tcgen05"),     # T_v = 12: one 16-channel group of values
])
def test_value_channel_pruning(name, S, L, B, lam_v, R, kernel):
    """App. D through the whole path: value scores and their ranking, thinned prefix values,
    tail values in the permuted order, decode over thinned keys AND values."""
    w = dataclasses.replace(wl.shrink(wl.get_config(name), S=S, L=L, B=B, steps=5), S_recent=R)
    data = wl.make_prefill(w, device="cpu")
    K, V, Q = data["K"].cuda(), data["V"].cuda(), data["Q_obs"].cuda()
    cache = make_cache(w, w.steps, lam_v=lam_v, value_score_kernel=1 if kernel == "mma_sync" else 0)
    cache.prefill(Q, K, V)
    torch.cuda.synchronize()
    o = make_oracle(w, lam_v)
    K64, V64, Q64 = to64(data["K"]), to64(data["V"]), to64(data["Q_obs"])
    o.score_select(Q64, K64)
    o.score_select_v(Q64, K64, V64)
    compare_selection(cache.idx_tensor().cpu().numpy(), cache.scores_tensor().cpu().numpy(), o, w.name)
    perm = cache.perm_v_tensor().cpu().numpy()
    assert (np.sort(perm, axis=-1) == np.arange(w.D)).all(), "perm_v must be a permutation"
    assert (np.diff(perm[..., o.T_v:].astype(np.int64), axis=-1) > 0).all()
    near = compare_selection(perm[..., : o.T_v], cache.scores_v_tensor().cpu().numpy(), o, w.name + " values",
                             values=True)
    record_parity(f"{w.name} value channels ({kernel})", near_ties=near, heads=w.B * w.L * w.N_kv)
    assert near <= max(1, (w.B * w.L * w.N_kv) // 4), f"{near} near-tie heads"
    o.compact(K64, V64)
    compare_cache(cache, o, where=w.name)
    for t in range(w.steps):
        st = wl.make_step(w, t, device="cpu")
        cache.append(st["k_new"].cuda(), st["v_new"].cuda())
        out = cache.decode_attn(st["q"].cuda())
        torch.cuda.synchronize()
        o.append(to64(st["k_new"]), to64(st["v_new"]))
        assert_attn_close(to64(out), o.decode_attn(to64(st["q"])), w.dtype, f"{w.name} step {t}")
    compare_cache(cache, o, where=w.name + " after decode")
    assert cache.device_error() == 0


def test_value_channel_pruning_state_and_support():
    from paper_2407_21018_b200 import binding as tk
    w = wl.shrink(wl.get_config("c2"), S=300, L=1, steps=2)
    data = wl.make_prefill(w, device="cuda")
    plain = make_cache(w, 2)
    with pytest.raises(tk.ThinKError) as e:              # no value pruning configured
        plain.score_select_kv(data["Q_obs"], data["K"], data["V"])
    assert e.value.status == tk.ERR_STATE
    kv = make_cache(w, 2, lam_v=0.5)
    kv.score_select(data["Q_obs"], data["K"])
    with pytest.raises(tk.ThinKError) as e:              # value channels not ranked yet
        kv.compact(data["K"], data["V"])
    assert e.value.status == tk.ERR_STATE
    kv.prefill(data["Q_obs"], data["K"], data["V"])
    with pytest.raises(tk.ThinKError) as e:
        kv.reprune_tail(0)
    assert e.value.status == tk.ERR_UNSUPPORTED
    w32 = wl.shrink(wl.get_config("c1"), S=100, steps=1)
    with pytest.raises(tk.ThinKError) as e:              # fp32 caches have no value-pruning kernels
        make_cache(w32, 1, lam_v=0.5)
    assert e.value.status == tk.ERR_UNSUPPORTED


@pytest.mark.parametrize("name,lam_v", [("c2", 0.0), ("c4", 0.0), ("c2", 0.3), ("c1", 0.0)])
def test_append_decode_in_one_call(name, lam_v):
    """thinK_append_decode (attention launched as a programmatic dependent of the append) gives bit-identical
    outputs and cache contents to thinK_append + thinK_decode_attn, step after step, and matches the oracle."""
    base = wl.get_config(name)
    w = wl.shrink(base, S=900, L=min(base.L, 2), B=min(base.B, 3), steps=70)
    data = wl.make_prefill(w, device="cuda")
    a, b = make_cache(w, w.steps, lam_v=lam_v), make_cache(w, w.steps, lam_v=lam_v)
    for c in (a, b):
        c.prefill(data["Q_obs"], data["K"], data["V"])
    o = make_oracle(w, lam_v)
    K64, V64, Q64 = to64(data["K"]), to64(data["V"]), to64(data["Q_obs"])
    o.score_select(Q64, K64)
    compare_selection(a.idx_tensor().cpu().numpy(), None, o, w.name)
    if lam_v > 0:
        o.score_select_v(Q64, K64, V64)
        compare_selection(a.perm_v_tensor().cpu().numpy()[..., : o.T_v], None, o, w.name + " values", values=True)
    o.compact(K64, V64)
    for t in range(w.steps):
        st = wl.make_step(w, t, device="cuda")
        a.append(st["k_new"], st["v_new"])
        out_a = a.decode_attn(st["q"])
        out_b = b.append_decode(st["k_new"], st["v_new"], st["q"])
        torch.cuda.synchronize()
        assert torch.equal(out_a, out_b), f"step {t}: fused step differs from the two calls"
        o.append(to64(st["k_new"]), to64(st["v_new"]))
        if t % 23 == 0 or t == w.steps - 1:
            assert_attn_close(to64(out_b), o.decode_attn(to64(st["q"])), w.dtype, f"{w.name} step {t}")
    from paper_2407_21018_b200 import binding as tk
    for (bb, l, h) in [(0, 0, 0), (w.B - 1, w.L - 1, w.N_kv - 1)]:
        ka, va = tk.tail_logical(a, bb, l, h)
        kb, vb = tk.tail_logical(b, bb, l, h)
        assert torch.equal(ka, kb) and torch.equal(va, vb)
    assert a.tail_len() == b.tail_len() == w.recent + w.steps
    assert b.device_error() == 0


@pytest.mark.parametrize("lam", [0.0, 0.25, 0.75])
def test_lambda_sweep(lam):
    w = wl.shrink(wl.get_config("c5"), S=1000, L=1, steps=3, lam=lam)
    run_case(w)


def test_lambda_zero_is_dense_attention():
    """lambda = 0 keeps every channel: the CUDA path must then equal plain dense attention."""
    w = wl.shrink(wl.get_config("c2"), S=777, L=1, steps=2, lam=0.0)
    r = run_case(w)
    o = r["oracle"]
    assert (o.idx == np.arange(w.D)).all()


@pytest.mark.parametrize("R", [0, 1, 128])
def test_recent_sizes(R):
    w = dataclasses.replace(wl.shrink(wl.get_config("c2"), S=600, L=1, steps=3), S_recent=R)
    run_case(w)


def test_all_tokens_recent():
    """S_recent = S: empty pruned prefix, everything lives in the unpruned tail."""
    w = wl.shrink(wl.get_config("c1"), S=96, steps=3)
    w = dataclasses.replace(w, S_recent=w.seq_lens[0])
    run_case(w)


def test_shortest_prompt():
    """S = S_obs + 1 (one pruned token) and S = S_obs with S_recent = 0."""
    w = wl.shrink(wl.get_config("c1"), S=33, steps=2)
    run_case(w)
    w = dataclasses.replace(wl.shrink(wl.get_config("c1"), S=33, steps=2), seq_lens=(32,), S_recent=0)
    run_case(w)


@pytest.mark.parametrize("dtype,D,G", [("f32", 128, 2), ("bf16", 64, 8), ("f32", 64, 1), ("bf16", 128, 1),
                                       ("bf16", 64, 2), ("f32", 128, 4)])
def test_shapes(dtype, D, G):
    w = wl.Workload("shape", dtype, 2, 2, 2 * G, 2, D, (300, 171), 16, 0.4, 3, 10000.0, (2, 10.0), 0x5EED + D + G)
    run_case(w)


@pytest.mark.parametrize("D,G,lam_v", [(64, 8, 0.5), (64, 2, 0.3), (128, 8, 0.3), (128, 2, 0.6)])
def test_value_channel_pruning_shapes(D, G, lam_v):
    """Value-channel pruning on the other head shapes: D = 64 (mma.sync score kernel), group sizes 2 and 8
    (S_obs = 16: 32 or 128 stacked window rows), ragged batch."""
    w = wl.Workload("vshape", "bf16", 2, 2, 2 * G, 2, D, (300, 171), 16, 0.4, 3, 10000.0, (2, 10.0), 0x5EED + D + G)
    data = wl.make_prefill(w, device="cpu")
    cache = make_cache(w, w.steps, lam_v=lam_v)
    cache.prefill(data["Q_obs"].cuda(), data["K"].cuda(), data["V"].cuda())
    o = make_oracle(w, lam_v)
    K64, V64, Q64 = to64(data["K"]), to64(data["V"]), to64(data["Q_obs"])
    o.score_select(Q64, K64)
    o.score_select_v(Q64, K64, V64)
    compare_selection(cache.idx_tensor().cpu().numpy(), cache.scores_tensor().cpu().numpy(), o, w.name)
    compare_selection(cache.perm_v_tensor().cpu().numpy()[..., : o.T_v], cache.scores_v_tensor().cpu().numpy(), o,
                      w.name + " values", values=True)
    o.compact(K64, V64)
    compare_cache(cache, o, where=w.name)
    for t in range(w.steps):
        st = wl.make_step(w, t, device="cpu")
        out = cache.append_decode(st["k_new"].cuda(), st["v_new"].cuda(), st["q"].cuda())
        torch.cuda.synchronize()
        o.append(to64(st["k_new"]), to64(st["v_new"]))
        assert_attn_close(to64(out), o.decode_attn(to64(st["q"])), w.dtype, f"{w.name} step {t}")
    assert cache.device_error() == 0


@pytest.mark.parametrize("criterion", [1, 2])
def test_magnitude_criteria(criterion):
    """Eq. 1 criteria (key l2 / l1 norms) through the same kernels."""
    w = wl.shrink(wl.get_config("c4"), S=500, L=1, B=2, steps=2)
    run_case(w, criterion=criterion)


def test_exact_ties_go_to_lower_channel():
    """Duplicate channels give exactly equal scores; the lower index must win on both sides."""
    w = wl.shrink(wl.get_config("c1"), S=200, steps=0)
    data = wl.make_prefill(w, device="cpu")
    K, Q = data["K"], data["Q_obs"]
    for a, b in ((3, 40), (7, 8), (10, 63)):
        K[..., b] = K[..., a]
        Q[..., b] = Q[..., a]
    cache = make_cache(w, 0)
    cache.score_select(Q.cuda(), K.cuda())
    torch.cuda.synchronize()
    o = make_oracle(w)
    o.score_select(to64(Q), to64(K))
    got = cache.idx_tensor().cpu().numpy().astype(np.int64)
    assert (got == o.idx).all()
    sc = cache.scores_tensor().cpu().numpy()
    assert (sc[..., 3] == sc[..., 40]).all()


def test_non_finite_keys_raise_the_error_word_and_stay_in_bounds():
    """A NaN in one key column makes that channel's score NaN.  The ranking must still keep exactly T
    channels per head (guard bytes behind every idx row survive) and the device error word must say so."""
    from paper_2407_21018_b200 import binding as tk
    w = wl.shrink(wl.get_config("c2"), S=500, L=2, steps=1)
    data = wl.make_prefill(w, device="cpu")
    K = data["K"].clone()
    K[0, 17, 1, 3, 40] = float("nan")                      # layer 1, key head 3, channel 40
    K[0, 18, 0, 5, 7] = float("inf")                       # layer 0, key head 5, channel 7
    cache = make_cache(w, 1)
    cache.idx.fill_(0xEE)
    cache.score_select(data["Q_obs"].cuda(), K.cuda())
    torch.cuda.synchronize()
    assert cache.device_error() & tk.ERR_BIT_NON_FINITE
    idx = cache.idx_tensor().cpu().numpy().astype(np.int64)
    assert (np.diff(idx, axis=-1) > 0).all() and idx.max() < w.D          # T distinct channels in every head
    n = w.B * w.L * w.N_kv * cache.T
    assert (cache.idx[n:] == 0xEE).all()                                    # nothing written past the last row
    assert 40 not in idx[0, 1, 3]                                           # the NaN channel ranks lowest
    assert 7 in idx[0, 0, 5]                                                # an infinite score ranks highest
    # untouched heads select what they select without the planted values
    ref = make_cache(w, 1)
    ref.score_select(data["Q_obs"].cuda(), data["K"].cuda())
    torch.cuda.synchronize()
    assert ref.device_error() == 0
    keep = np.ones((w.L, w.N_kv), dtype=bool)
    keep[1, 3] = keep[0, 5] = False
    assert (idx[0][keep] == ref.idx_tensor().cpu().numpy().astype(np.int64)[0][keep]).all()


def test_layer_ranges_and_determinism():
    """Per-layer calls give the same bytes as one call over all layers, and a repeat is identical."""
    w = wl.shrink(wl.get_config("c2"), S=900, L=3, steps=2)
    data = wl.make_prefill(w, device="cpu")
    K, V, Q = data["K"].cuda(), data["V"].cuda(), data["Q_obs"].cuda()
    a, b = make_cache(w, 2), make_cache(w, 2)
    a.score_select(Q, K)
    a.compact(K, V)
    for l in (2, 0, 1):
        b.score_select(Q, K, layer0=l, nlayers=1)
        b.compact(K, V, layer0=l, nlayers=1)
    torch.cuda.synchronize()
    assert torch.equal(a.idx_tensor(), b.idx_tensor())
    n = a.sizes.k_thin
    assert torch.equal(a.k_thin[:n], b.k_thin[:n])
    st = wl.make_step(w, 0, device="cuda")
    a.append(st["k_new"], st["v_new"])
    out_a = a.decode_attn(st["q"])
    out_a2 = a.decode_attn(st["q"])
    outs = []
    for l in range(3):
        b.append(st["k_new"][:, l:l + 1].contiguous(), st["v_new"][:, l:l + 1].contiguous(), layer0=l, nlayers=1)
        outs.append(b.decode_attn(st["q"][:, l:l + 1].contiguous(), layer0=l, nlayers=1))
    torch.cuda.synchronize()
    assert torch.equal(out_a, out_a2)
    got = torch.cat(outs, dim=1)
    # split boundaries differ between the two launch shapes: same values up to fp32 merge order
    assert (got.float() - out_a.float()).abs().max().item() <= 1e-2


def test_strided_per_layer_cache_layout():
    """A [B, N, S, D]-per-layer cache expressed through the strides of the 5-d view."""
    w = wl.shrink(wl.get_config("c2"), S=500, L=2, steps=2)
    data = wl.make_prefill(w, device="cpu")
    perm = lambda t: t.permute(2, 0, 3, 1, 4).contiguous().permute(1, 3, 0, 2, 4)   # storage [L, B, N, S, D]
    Kc, Vc, Qc = data["K"].cuda(), data["V"].cuda(), data["Q_obs"].cuda()
    a, b = make_cache(w, 2), make_cache(w, 2)
    K, V, Q = perm(Kc), perm(Vc), perm(Qc)
    assert K.stride(1) == w.D
    a.score_select(Q, K)
    a.compact(K, V)
    b.score_select(Qc, Kc)
    b.compact(Kc, Vc)
    st = wl.make_step(w, 0, device="cuda")
    for c in (a, b):
        c.append(st["k_new"], st["v_new"])
    oa, ob = a.decode_attn(st["q"]), b.decode_attn(st["q"])
    torch.cuda.synchronize()
    assert torch.equal(a.idx_tensor(), b.idx_tensor())
    assert torch.equal(a.k_thin, b.k_thin)
    assert torch.equal(oa, ob)


def test_state_machine_and_capacity():
    from paper_2407_21018_b200 import binding as tk
    w = wl.shrink(wl.get_config("c1"), S=128, steps=2)
    data = wl.make_prefill(w, device="cuda")
    c = make_cache(w, 2)
    st = wl.make_step(w, 0, device="cuda")
    with pytest.raises(tk.ThinKError) as e:
        c.compact(data["K"], data["V"])
    assert e.value.status == tk.ERR_STATE
    with pytest.raises(tk.ThinKError) as e:
        c.append(st["k_new"], st["v_new"])
    assert e.value.status == tk.ERR_STATE
    with pytest.raises(tk.ThinKError) as e:
        c.decode_attn(st["q"])
    assert e.value.status == tk.ERR_STATE
    with pytest.raises(tk.ThinKError) as e:
        c.score_select(data["Q_obs"], data["K"], layer0=1, nlayers=1)
    assert e.value.status == tk.ERR_INVALID_ARG
    c.score_select(data["Q_obs"], data["K"])
    c.compact(data["K"], data["V"])
    assert c.tail_len() == w.recent
    c.append(st["k_new"], st["v_new"])
    c.append(st["k_new"], st["v_new"])
    with pytest.raises(tk.ThinKError) as e:
        c.append(st["k_new"], st["v_new"])
    assert e.value.status == tk.ERR_CAPACITY
    assert c.tail_len() == w.recent + 2
    torch.cuda.synchronize()
    assert c.device_error() == 0


def test_new_prompt_on_the_same_handle_reborrows_the_values():
    """A second prefill with a different V view is a new prompt: it is accepted, the layers it does not cover
    count as not compacted until they are, and decode then reads the NEW values."""
    from paper_2407_21018_b200 import binding as tk
    w = wl.shrink(wl.get_config("c2"), S=700, L=2, steps=2)
    data = wl.make_prefill(w, device="cuda")
    K, V, Q = data["K"], data["V"], data["Q_obs"]
    st = wl.make_step(w, 0, device="cuda")
    c = make_cache(w, 2)
    c.prefill(Q, K, V)
    V2 = (V.float() * 0.5).to(V.dtype)                      # same shape, other storage, other numbers
    c.prefill(Q, K, V2, layer0=0, nlayers=1)                # covers layer 0 only
    with pytest.raises(tk.ThinKError) as e:
        c.append(st["k_new"], st["v_new"])                  # layer 1 still belongs to the old prompt
    assert e.value.status == tk.ERR_STATE
    c.prefill(Q, K, V2, layer0=1, nlayers=1)
    c.append(st["k_new"], st["v_new"])
    out = c.decode_attn(st["q"])
    fresh = make_cache(w, 2)
    fresh.prefill(Q, K, V2)
    fresh.append(st["k_new"], st["v_new"])
    want = fresh.decode_attn(st["q"])
    torch.cuda.synchronize()
    assert torch.equal(out, want)
    assert c.device_error() == 0


def test_guard_bytes_untouched():
    """Outputs stay inside their buffers: canaries after out / idx survive."""
    w = wl.shrink(wl.get_config("c4"), S=300, L=1, B=3, steps=1)
    data = wl.make_prefill(w, device="cuda")
    c = make_cache(w, 1)
    c.score_select(data["Q_obs"], data["K"])
    c.compact(data["K"], data["V"])
    st = wl.make_step(w, 0, device="cuda")
    c.append(st["k_new"], st["v_new"])
    n = st["q"].numel()
    buf = torch.full((n + 64,), 7.0, dtype=st["q"].dtype, device="cuda")
    c.decode_attn(st["q"], out=buf[:n].view_as(st["q"]))
    torch.cuda.synchronize()
    assert (buf[n:] == 7.0).all()
    assert torch.isfinite(buf[:n].float()).all()


def _sampled_full_size(name, units, steps_checked, lam=None, lam_v=0.0):
    """Full-size workload in the launch configuration the benchmark times; the oracle checks
    sampled (b, layer, key head) units: literal + closed-form scores, selection, compacted keys and
    the attention rows of the unit's query heads."""
    w = wl.get_config(name)
    if lam is not None:
        w = dataclasses.replace(w, lam=lam)
    data = wl.make_prefill(w, device="cuda")
    K, V, Q = data["K"], data["V"], data["Q_obs"]
    cache = make_cache(w, max(steps_checked) + 1, lam_v=lam_v)
    cache.prefill(Q, K, V)           # the launch configuration the benchmark times
    torch.cuda.synchronize()
    assert cache.device_error() == 0
    from paper_2407_21018_b200 import binding as tk
    G = w.N_q // w.N_kv
    idx_gpu = cache.idx_tensor().cpu().numpy().astype(np.int64)
    sc_gpu = cache.scores_tensor().cpu().numpy()
    heads = {}
    for n, (b, l, h) in enumerate(units):
        S_b = w.seq_lens[b]
        Kh, Vh = to64(K[b, :S_b, l, h]), to64(V[b, :S_b, l, h])
        Qg = np.stack([to64(Q[b, :, l, h * G + g]) for g in range(G)])
        s = orc.score_closed_form(Qg, Kh)
        if n == 0:
            np.testing.assert_allclose(orc.score_literal(Qg, Kh), s, rtol=1e-12)
        np.testing.assert_allclose(sc_gpu[b, l, h], s, rtol=1e-6)
        check_head_selection(idx_gpu[b, l, h], s, cache.T, NEAR_TIE_REL, f"{name} {(b, l, h)}")
        idx = idx_gpu[b, l, h]              # the oracle's choice, or its near-tie alternative
        K_T, K_r = orc.compact_keys(Kh, idx, w.recent)
        assert (to64(tk.k_thin_logical(cache, b, l, h)) == K_T).all()
        heads[(b, l, h)] = dict(idx=idx, K_T=K_T, K_full=K_r, V=Vh)
        if lam_v > 0:                # value channels (App. D): scores, ranking, thinned prefix rows
            sv = orc.score_value(Qg, Kh, Vh)
            np.testing.assert_allclose(cache.scores_v_tensor()[b, l, h].cpu().numpy(), sv, rtol=1e-4)
            perm = cache.perm_v_tensor()[b, l, h].cpu().numpy().astype(np.int64)
            assert (np.sort(perm) == np.arange(w.D)).all()
            check_head_selection(perm[: cache.T_v], sv, cache.T_v, NEAR_TIE_V_REL, f"{name} values {(b, l, h)}")
            idx_v = perm[: cache.T_v]
            S_p = S_b - w.recent
            assert (to64(tk.v_thin_logical(cache, b, l, h)) == Vh[:S_p][:, idx_v]).all()
            heads[(b, l, h)].update(idx_v=idx_v, V_T=Vh[:S_p][:, idx_v], V=Vh[S_p:])
    worst = 0.0
    for t in range(max(steps_checked) + 1):
        st = wl.make_step(w, t, device="cuda")
        cache.append(st["k_new"], st["v_new"])
        out = cache.decode_attn(st["q"])
        torch.cuda.synchronize()
        for (b, l, h), d in heads.items():
            d["K_full"] = np.vstack([d["K_full"], to64(st["k_new"][b, l, h])[None]])
            d["V"] = np.vstack([d["V"], to64(st["v_new"][b, l, h])[None]])
            if t in steps_checked:
                for g in range(G):
                    qrow = to64(st["q"][b, l, h * G + g])
                    if lam_v > 0:
                        want = orc.decode_attention_kv(qrow, d["K_T"], d["idx"], d["K_full"], d["V_T"], d["idx_v"], d["V"])
                    else:
                        want = orc.decode_attention(qrow, d["K_T"], d["idx"], d["K_full"], d["V"])
                    worst = max(worst, assert_attn_close(to64(out[b, l, h * G + g]), want, w.dtype, f"{name} {(b, l, h, g)} t={t}"))
        if t in steps_checked:
            assert torch.isfinite(out.float()).all()
    assert cache.device_error() == 0
    return worst


def test_c2_full_size_sampled_value_pruning():
    _sampled_full_size("c2", [(0, 0, 0), (0, 19, 6), (0, 31, 3)], {0, 2}, lam_v=0.3)


def test_c4_full_size_sampled_value_pruning():
    _sampled_full_size("c4", [(0, 0, 0), (15, 31, 31), (9, 20, 4)], {0, 1}, lam_v=0.5)


def test_c5_full_size_sampled_value_pruning():
    _sampled_full_size("c5", [(0, 17, 4)], {0}, lam_v=0.5)
