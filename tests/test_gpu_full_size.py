"""Full-size parity of configs c2-c5, in the launch configuration the benchmark times.

Per config, against the CPU oracle on the same seeded inputs:
  * channel scores (rtol 1e-6) and Top_T for EVERY (batch entry, layer, key head): the closed-form oracle
    score, head by head, on key slabs downloaded from the device; the literal Frobenius-norm score on one
    head; indices bit-exact, near-ties (oracle scores at the cut closer than 1e-6 relative, disagreement
    confined to that band) counted;
  * compacted keys and the seeded tail bit-exact on every head of c2 and on 64 spread heads of c3-c5;
  * attention at the first and at the LAST decode step of the config (the longest tail) for all heads of c2
    and 32 spread heads of c3-c5, within 1e-2 max-abs;
  * c5 at lambda in {0, 0.25, 0.75} on sampled heads.
Statistics (near-ties, max-abs error, outputs of magnitude >= 4, which take the half-ulp bar) go to the
end-of-run summary."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import think_oracle as orc
from paper_2407_21018_b200 import workloads as wl

from _harness import (NEAR_TIE_REL, SCORE_RTOL, assert_attn_close, check_head_selection, make_cache, record_parity, to64)

pytestmark = pytest.mark.gpu

_DATA = {}


def _prefill_data(name):
    """One set of prompt tensors per config at a time (they are 17-26 GB each)."""
    if name not in _DATA:
        _DATA.clear()
        torch.cuda.empty_cache()
        _DATA[name] = wl.make_prefill(wl.get_config(name), device="cuda")
    return _DATA[name]


def _spread(w, count):
    """`count` distinct (b, l, h) units spread over the whole range, first and last included."""
    total = w.B * w.L * w.N_kv
    picks = sorted({int(round(i * (total - 1) / max(1, count - 1))) for i in range(count)}) if count < total else range(total)
    return [(u // (w.L * w.N_kv), (u // w.N_kv) % w.L, u % w.N_kv) for u in picks]


def _full_size(name, n_cache_units, n_attn_units, steps_checked, lam=None, all_heads=True):
    from paper_2407_21018_b200 import binding as tk
    w = wl.get_config(name)
    data = _prefill_data(name)
    if lam is not None:
        w = dataclasses.replace(w, lam=lam, name=f"{name}-lam{lam}")
    K, V, Q = data["K"], data["V"], data["Q_obs"]
    last = max(steps_checked)
    cache = make_cache(w, last + 1)
    cache.prefill(Q, K, V)                      # the call the benchmark times
    torch.cuda.synchronize()
    assert cache.device_error() == 0
    G, T, R = w.N_q // w.N_kv, cache.T, w.recent
    idx_gpu = cache.idx_tensor().cpu().numpy().astype(np.int64)
    sc_gpu = cache.scores_tensor().cpu().numpy()
    cache_units = set(_spread(w, n_cache_units))
    attn_units = _spread(w, n_attn_units)
    heads = {}
    near = mism = checked = 0
    literal_done = False
    sel_units = [(b, l) for b in range(w.B) for l in range(w.L)] if all_heads else sorted({(b, l) for (b, l, _) in cache_units | set(attn_units)})
    for (b, l) in sel_units:
        S_b = w.seq_lens[b]
        # one (b, layer) slab of keys, widened exactly to fp64, head-major
        Ks = np.ascontiguousarray(K[b, :S_b, l].to(torch.float64).cpu().numpy().transpose(1, 0, 2))   # [N_kv, S_b, D]
        Qs = Q[b, :, l].to(torch.float64).cpu().numpy()                                                # [S_obs, N_q, D]
        for h in range(w.N_kv):
            if not all_heads and (b, l, h) not in cache_units and (b, l, h) not in attn_units:
                continue
            Qg = np.stack([Qs[:, h * G + g, :] for g in range(G)])
            s = orc.score_closed_form(Qg, Ks[h])
            if not literal_done:
                np.testing.assert_allclose(orc.score_literal(Qg, Ks[h]), s, rtol=1e-12)
                literal_done = True
            np.testing.assert_allclose(sc_gpu[b, l, h], s, rtol=SCORE_RTOL, err_msg=f"{w.name} scores at {(b, l, h)}")
            tie = check_head_selection(idx_gpu[b, l, h], s, T, NEAR_TIE_REL, f"{w.name} {(b, l, h)}")
            near += tie
            mism += int(tie and not (idx_gpu[b, l, h] == orc.select_top_T(s, T)).all())
            checked += 1
            idx = idx_gpu[b, l, h]              # identical to the oracle's, or its near-tie alternative
            if (b, l, h) in cache_units or (b, l, h) in attn_units:
                K_T, K_r = orc.compact_keys(Ks[h], idx, R)
                assert (to64(tk.k_thin_logical(cache, b, l, h)) == K_T).all(), f"{w.name} K_T differs at {(b, l, h)}"
                kf, vf = tk.tail_logical(cache, b, l, h)
                assert (to64(kf) == K_r).all(), f"{w.name} tail keys differ at {(b, l, h)}"
                Vh = to64(V[b, :S_b, l, h])
                assert (to64(vf) == Vh[S_b - R:]).all(), f"{w.name} tail values differ at {(b, l, h)}"
                if (b, l, h) in attn_units:
                    heads[(b, l, h)] = dict(idx=idx, K_T=K_T, K_new=[K_r], V_new=[Vh])
    # decode up to the last step; the oracle sees the sampled heads' new rows
    stats = {}
    ub = torch.tensor([u[0] for u in attn_units], device="cuda")
    ul = torch.tensor([u[1] for u in attn_units], device="cuda")
    uh = torch.tensor([u[2] for u in attn_units], device="cuda")
    for t in range(last + 1):
        st = wl.make_step(w, t, device="cuda")
        cache.append(st["k_new"], st["v_new"])
        kn, vn = to64(st["k_new"][ub, ul, uh]), to64(st["v_new"][ub, ul, uh])
        for n, u in enumerate(attn_units):
            heads[u]["K_new"].append(kn[n][None])
            heads[u]["V_new"].append(vn[n][None])
        if t not in steps_checked:
            continue
        out = cache.decode_attn(st["q"])
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        qs = torch.stack([st["q"][ub, ul, uh * G + g] for g in range(G)], dim=1)      # [units, G, D]
        got = torch.stack([out[ub, ul, uh * G + g] for g in range(G)], dim=1)
        qs, got = to64(qs), to64(got)
        for n, u in enumerate(attn_units):
            d = heads[u]
            K_full, V_all = np.vstack(d["K_new"]), np.vstack(d["V_new"])
            for g in range(G):
                want = orc.decode_attention(qs[n, g], d["K_T"], d["idx"], K_full, V_all)
                assert_attn_close(got[n, g], want, w.dtype, f"{w.name} {u} g={g} t={t}", stats)
    assert cache.device_error() == 0
    record_parity(w.name + " full size", heads_selected=checked, near_ties=near, idx_mismatches=mism,
                  heads_cache_exact=len(cache_units | set(attn_units)), heads_attention=len(attn_units),
                  steps=sorted(steps_checked), max_abs=stats.get("max_abs"), outputs_ge_4=stats.get("large", 0))
    del cache
    torch.cuda.empty_cache()


def test_c2_full_size_every_head():
    w = wl.get_config("c2")
    _full_size("c2", w.L * w.N_kv, w.L * w.N_kv, {0, w.steps - 1})


def test_c3_full_size():
    w = wl.get_config("c3")
    _full_size("c3", 64, 32, {0, w.steps - 1})


def test_c4_full_size():
    w = wl.get_config("c4")
    _full_size("c4", 64, 32, {0, w.steps - 1})


def test_c5_full_size():
    w = wl.get_config("c5")
    _full_size("c5", 64, 32, {0, w.steps - 1})


@pytest.mark.parametrize("lam", [0.0, 0.25, 0.75])
def test_c5_full_size_lambda_sweep(lam):
    _full_size("c5", 6, 4, {0, 2}, lam=lam, all_heads=False)


def test_release_prompt_tensors():
    _DATA.clear()
    torch.cuda.empty_cache()
