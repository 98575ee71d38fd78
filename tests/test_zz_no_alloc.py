"""thinK_score_select_static -- the entry point for callers that may not allocate device memory
(plugins living inside someone else's memory pool, fixed-budget processes): the library's own
built-in scratch replaces the caller-allocated workspace.  Checked here against the regular
thinK_score_select on the same inputs: selected channels identical, scores to 1e-12 relative
(the two calls may split the tokens differently, which reorders fp64 sums).  Two calls in a row on
different data, so the second one runs on a scratch array that still holds the first one's state."""
import numpy as np
import pytest
import torch

from paper_2407_21018_b200 import workloads as wl

from _harness import make_cache

pytestmark = pytest.mark.gpu


def _both(w, rtol=1e-12):
    from paper_2407_21018_b200 import binding as tk
    data = wl.make_prefill(w, device="cuda")
    ref = make_cache(w, 1)
    ref.score_select(data["Q_obs"], data["K"])
    idx = torch.full((w.B, w.L, w.N_kv, ref.T), 255, dtype=torch.uint8, device="cuda")
    scores = torch.full((w.B, w.L, w.N_kv, w.D), -1.0, dtype=torch.float64, device="cuda")
    tk.score_select_static(ref.cfg, w.seq_lens, data["Q_obs"], data["K"], idx, scores)
    torch.cuda.synchronize()
    assert torch.equal(idx, ref.idx_tensor())
    np.testing.assert_allclose(scores.cpu().numpy(), ref.scores_tensor().cpu().numpy(), rtol=rtol)


def test_static_scratch_entry_matches_regular_entry_twice():
    _both(wl.shrink(wl.get_config("c2"), S=3000, L=3))                       # GQA, bf16
    _both(wl.shrink(wl.get_config("c4"), S=900, L=2, B=4))                   # MHA, ragged, two column blocks
    _both(wl.shrink(wl.get_config("c1"), S=300))                             # fp32


def test_static_scratch_entry_lowers_its_token_split_to_fit():
    """16 sequences-times-layers-times-column-blocks items of 32 KB partials each: the token split the call would
    like (7) needs more than the 8 MiB array, so it settles for 5.  Same channels; the scores agree to the
    tolerance the parity tests give a score (1e-6): another split regroups the fp32 chains of 8 squares."""
    _both(wl.shrink(wl.get_config("c4"), S=900, L=6, B=4), rtol=1e-6)


def test_static_scratch_entry_allocates_nothing():
    """Free device memory (as the driver reports it) is the same before and after a call: no cudaMalloc
    behind the caller's back.  The first call, which looks up the array's address, has already happened."""
    from paper_2407_21018_b200 import binding as tk
    w = wl.shrink(wl.get_config("c2"), S=2000, L=2)
    data = wl.make_prefill(w, device="cuda")
    cfg = tk.make_config(w.B, w.L, w.N_q, w.N_kv, w.D, w.S_max, w.S_obs, w.recent, 1, w.lam, w.torch_dtype)
    idx = torch.zeros((w.B, w.L, w.N_kv, tk.thinK_T(w.lam, w.D)), dtype=torch.uint8, device="cuda")
    tk.score_select_static(cfg, w.seq_lens, data["Q_obs"], data["K"], idx)      # address lookup done at the latest here
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        tk.score_select_static(cfg, w.seq_lens, data["Q_obs"], data["K"], idx)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_static_scratch_entry_rejects_oversize():
    from paper_2407_21018_b200 import binding as tk
    w = wl.get_config("c4")          # 16 x 32 layers x 4096 columns of fp64 partials: far beyond 8 MiB
    cfg = tk.make_config(w.B, w.L, w.N_q, w.N_kv, w.D, w.S_max, w.S_obs, w.recent, 1, w.lam, w.torch_dtype)
    k = torch.zeros((1, 1, 1, 1, w.D), dtype=torch.bfloat16, device="cuda").expand(w.B, w.S_max, w.L, w.N_kv, w.D)
    idx = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(tk.ThinKError) as e:
        tk.score_select_static(cfg, w.seq_lens, k, k, idx)        # refused before anything is launched
    assert e.value.status == tk.ERR_CAPACITY
