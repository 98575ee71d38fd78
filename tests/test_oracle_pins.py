"""Pins for the CPU oracle: each test ties one oracle routine to something other
than itself -- a closed form, a brute-force search, a special case that reduces
to textbook attention, a hand-computed example, or a figure the paper prints."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import think_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([float(x) for x in line.split()])
    return out


# ------------------------------------------------------------------ T
def test_kept_channels_values():
    # Sec. 3.1: T = floor((1 - lambda) D); values for the five workloads
    assert orc.kept_channels(0.5, 64) == 32
    assert orc.kept_channels(0.4, 128) == 76      # 76.8 floors to 76
    assert orc.kept_channels(0.5, 128) == 64
    assert orc.kept_channels(0.6, 128) == 51      # 51.2
    assert orc.kept_channels(0.0, 128) == 128
    assert orc.kept_channels(0.25, 128) == 96
    assert orc.kept_channels(0.75, 128) == 32
    assert orc.kept_channels(0.4, 5) == 3         # (1 - 0.4) * 5 is 2.9999999999999996 in binary
    with pytest.raises(ValueError):
        orc.kept_channels(1.0, 64)
    with pytest.raises(ValueError):
        orc.kept_channels(0.999, 64)


# ------------------------------------------------------------------ score
def test_score_hand_example():
    # one channel: q column (3, 4), k column (1, 2, 2): outer product has
    # Frobenius norm 5 * 3 = 15; second channel q (1, 0), k (0, 0, 7) -> 7
    Q = np.array([[[3.0, 1.0], [4.0, 0.0]]])          # [G=1, S_obs=2, D=2]
    K = np.array([[1.0, 0.0], [2.0, 0.0], [2.0, 7.0]])
    np.testing.assert_allclose(orc.score_literal(Q, K), [15.0, 7.0], rtol=1e-15)
    np.testing.assert_allclose(orc.score_closed_form(Q, K), [15.0, 7.0], rtol=1e-15)


@pytest.mark.parametrize("G,S_obs,S,D", [(1, 4, 9, 6), (4, 8, 33, 16), (2, 32, 200, 64)])
def test_score_literal_equals_rank_one_identity(G, S_obs, S, D):
    rng = np.random.default_rng(7 + G + S)
    Q = rng.normal(size=(G, S_obs, D)) * np.exp(rng.normal(size=D))
    K = rng.normal(size=(S, D)) * np.exp(rng.normal(size=D))
    a = orc.score_literal(Q, K)
    b = orc.score_closed_form(Q, K)
    np.testing.assert_allclose(a, b, rtol=1e-12)
    # third route: Frobenius norm from the singular values of the interaction matrix
    j = D // 2
    M = np.outer(Q.reshape(-1, D)[:, j], K[:, j])
    assert abs(np.linalg.norm(np.linalg.svd(M, compute_uv=False)) - a[j]) <= 1e-12 * a[j]


def test_score_is_eq2_loss_for_one_pruned_channel():
    # Eq. 2 with exactly one channel pruned: the loss IS that channel's score,
    # so the channel greedy pruning drops first is the brute-force minimiser.
    rng = np.random.default_rng(3)
    G, S_obs, S, D = 2, 5, 17, 7
    Q = rng.normal(size=(G, S_obs, D)) * np.exp(rng.normal(size=D))
    K = rng.normal(size=(S, D)) * np.exp(rng.normal(size=D))
    s = orc.score_literal(Q, K)
    Qs = Q.reshape(-1, D)
    losses = []
    for j in range(D):
        keep = [c for c in range(D) if c != j]
        losses.append(orc.pruning_loss(Qs, K, keep))
    np.testing.assert_allclose(losses, s, rtol=1e-12)
    idx = orc.select_top_T(s, D - 1)
    dropped = (set(range(D)) - set(idx.tolist())).pop()
    assert dropped == int(np.argmin(losses))


def test_pruning_loss_independent_formula():
    # || Q K^T - Q S K^T ||_F^2 = sum over entries of (sum over pruned channels q k)^2
    rng = np.random.default_rng(11)
    Q = rng.normal(size=(4, 5))
    K = rng.normal(size=(6, 5))
    keep = [0, 3]
    acc = 0.0
    for s in range(4):
        for t in range(6):
            acc += sum(Q[s, c] * K[t, c] for c in (1, 2, 4)) ** 2
    assert abs(orc.pruning_loss(Q, K, keep) - math.sqrt(acc)) < 1e-12


def test_score_invariances():
    rng = np.random.default_rng(5)
    Q = rng.normal(size=(1, 8, 12))
    K = rng.normal(size=(40, 12)) * np.exp(rng.normal(size=12))
    T = 5
    base = orc.select_top_T(orc.score_closed_form(Q, K), T)
    perm = rng.permutation(40)                       # token order of K does not matter
    assert (orc.select_top_T(orc.score_closed_form(Q, K[perm]), T) == base).all()
    assert (orc.select_top_T(orc.score_closed_form(3.5 * Q, K), T) == base).all()
    assert (orc.select_top_T(orc.score_closed_form(Q, 0.25 * K), T) == base).all()


def test_cache_elements_with_decoded_tokens_hand_value():
    # Sec. 3.3 by hand: one head, D = 4, half the channels kept, a prompt of 10 tokens of which the last 2 stay
    # unpruned, 3 tokens decoded.  Keys: 8 pruned rows x 2 channels + (2 + 3) full rows x 4 = 16 + 20 = 36;
    # values: (10 + 3) rows x 4 = 52; total 88.  Two layers of three heads: x 6 = 528.
    assert orc.think_cache_elements([10], 1, 1, 4, keep=0.5, S_recent=2, new_tokens=3) == 88.0
    assert orc.think_cache_elements([10], 2, 3, 4, keep=0.5, S_recent=2, new_tokens=3) == 528.0
    # two sequences add up; without decoded tokens the tail holds the recent rows only
    assert orc.think_cache_elements([10, 6], 1, 1, 4, keep=0.5, S_recent=2, new_tokens=0) == (16 + 8 + 40) + (8 + 8 + 24)


def test_gqa_group_is_stacked_rows():
    # declared reading: the group's query heads are stacked; equals sqrt of summed squares
    rng = np.random.default_rng(9)
    Q = rng.normal(size=(4, 6, 10))
    K = rng.normal(size=(21, 10))
    per_head = np.stack([orc.score_literal(Q[g:g + 1], K) for g in range(4)])
    np.testing.assert_allclose(orc.score_literal(Q, K), np.sqrt((per_head ** 2).sum(0)), rtol=1e-12)


def test_magnitude_score_matches_library_norm():
    rng = np.random.default_rng(2)
    K = rng.normal(size=(31, 9))
    for p in (1, 2):
        np.testing.assert_allclose(orc.score_magnitude(K, p), np.linalg.norm(K, ord=p, axis=0), rtol=1e-13)


def test_magnitude_score_hand_values():
    # Eq. 1 on a 3 x 2 matrix worked by hand: column 0 = (3, -4, 0), column 1 = (1, 2, -2)
    K = np.array([[3.0, 1.0], [-4.0, 2.0], [0.0, -2.0]])
    assert orc.score_magnitude(K, 1).tolist() == [7.0, 5.0]        # |3| + |-4| + 0, 1 + 2 + 2
    assert orc.score_magnitude(K, 2).tolist() == [5.0, 3.0]        # sqrt(9 + 16), sqrt(1 + 4 + 4)
    # a transposed operand or a norm over the wrong axis gives (4, 6, 2) / (sqrt 10, sqrt 20, 2) instead


# ------------------------------------------------------------------ top-T
@pytest.mark.parametrize("D,T", [(5, 2), (8, 3), (10, 5), (12, 4)])
def test_topT_brute_force(D, T):
    rng = np.random.default_rng(100 + D)
    for _ in range(20):
        s = np.abs(rng.normal(size=D))
        best = max(itertools.combinations(range(D), T), key=lambda c: sum(s[list(c)]))
        assert tuple(orc.select_top_T(s, T)) == tuple(sorted(best))


def test_topT_ties_go_to_lower_index_and_edges():
    s = np.array([1.0, 3.0, 3.0, 0.5, 3.0, 2.0])
    assert orc.select_top_T(s, 1).tolist() == [1]
    assert orc.select_top_T(s, 2).tolist() == [1, 2]
    assert orc.select_top_T(s, 3).tolist() == [1, 2, 4]
    assert orc.select_top_T(s, 4).tolist() == [1, 2, 4, 5]
    assert orc.select_top_T(s, 6).tolist() == [0, 1, 2, 3, 4, 5]          # T = D: identity
    assert orc.select_top_T(np.array([0.1, 9.0, 0.3]), 1).tolist() == [1]  # T = 1: arg-max
    assert orc.select_top_T(np.zeros(4), 2).tolist() == [0, 1]            # all equal
    # duplicated channel: the copy with the lower index is kept first
    s = np.array([5.0, 2.0, 7.0, 2.0, 1.0])
    assert orc.select_top_T(s, 3).tolist() == [0, 1, 2]


def test_near_tie_flag():
    s = np.array([4.0, 3.0, 3.0 * (1 - 1e-8), 1.0])
    assert orc.near_tie(s, 2)
    assert not orc.near_tie(s, 1)
    assert not orc.near_tie(s, 3)


# ------------------------------------------------------------------ compaction
def test_compact_is_a_gather_and_scatters_back():
    rng = np.random.default_rng(4)
    K = rng.normal(size=(20, 8))
    idx = np.array([1, 2, 5, 7])
    K_T, K_r = orc.compact_keys(K, idx, 6)
    assert K_T.shape == (14, 4) and K_r.shape == (6, 8)
    back = np.zeros((14, 8))
    back[:, idx] = K_T
    assert (back[:, idx] == K[:14][:, idx]).all()
    assert (back[:, [0, 3, 4, 6]] == 0).all()
    assert (K_r == K[14:]).all()
    K_T0, K_r0 = orc.compact_keys(K, idx, 0)
    assert K_T0.shape == (20, 4) and K_r0.shape == (0, 8)


# ------------------------------------------------------------------ decode attention
def _dense_by_loops(q, K, V):
    """Textbook softmax attention written with scalar loops (separate from the oracle)."""
    D = len(q)
    x = [sum(q[c] * K[t][c] for c in range(D)) / math.sqrt(D) for t in range(len(K))]
    m = max(x)
    e = [math.exp(v - m) for v in x]
    Z = sum(e)
    return [sum(e[t] / Z * V[t][d] for t in range(len(K))) for d in range(len(V[0]))]


def test_decode_hand_example():
    # D = 2, channel 1 pruned.  Prefix of two tokens, one unpruned recent token.
    # q = (sqrt2 * ln2, 5): prefix logits use channel 0 only:
    #   k_T = 1 -> ln 2 ; k_T = 0 -> 0 ; recent key (0, 0) -> 0.
    # softmax(ln2, 0, 0) = (1/2, 1/4, 1/4); V = (4, 0), (0, 8), (8, 8) -> (4, 4)
    q = np.array([math.sqrt(2.0) * math.log(2.0), 5.0])
    K_T = np.array([[1.0], [0.0]])
    idx = np.array([0])
    K_full = np.array([[0.0, 0.0]])
    V = np.array([[4.0, 0.0], [0.0, 8.0], [8.0, 8.0]])
    np.testing.assert_allclose(orc.decode_attention(q, K_T, idx, K_full, V), [4.0, 4.0], rtol=1e-14)
    # the pruned channel of the query must not reach the prefix: with the
    # channel restored (recent-only cache) the same inputs give another answer
    K = np.array([[1.0, 3.0], [0.0, -3.0], [0.0, 0.0]])
    full = orc.decode_attention(q, np.zeros((0, 1)), idx, K, V)
    assert abs(full[1] - 4.0) > 1.0


def test_decode_single_token_is_its_value_row():
    q = np.array([0.3, -2.0, 1.0])
    out = orc.decode_attention(q, np.zeros((0, 2)), np.array([0, 2]), np.array([[1.0, 2.0, 3.0]]),
                               np.array([[7.0, -1.0, 0.5]]))
    np.testing.assert_allclose(out, [7.0, -1.0, 0.5], rtol=0, atol=0)


@pytest.mark.parametrize("S,D,R", [(13, 6, 0), (40, 16, 5), (70, 8, 32)])
def test_lambda_zero_is_dense_attention(S, D, R):
    rng = np.random.default_rng(S)
    q = rng.normal(size=D)
    K = rng.normal(size=(S, D)) * np.exp(rng.normal(size=D))
    V = rng.normal(size=(S, D))
    idx = orc.select_top_T(rng.random(D), orc.kept_channels(0.0, D))
    assert idx.tolist() == list(range(D))
    K_T, K_r = orc.compact_keys(K, idx, R)
    out = orc.decode_attention(q, K_T, idx, K_r, V)
    np.testing.assert_allclose(out, orc.dense_attention(q, K, V), rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(out, _dense_by_loops(q.tolist(), K.tolist(), V.tolist()), rtol=1e-12, atol=1e-13)


def test_all_recent_is_dense_for_any_lambda():
    rng = np.random.default_rng(8)
    S, D = 25, 12
    q, K, V = rng.normal(size=D), rng.normal(size=(S, D)), rng.normal(size=(S, D))
    idx = orc.select_top_T(rng.random(D), orc.kept_channels(0.5, D))
    K_T, K_r = orc.compact_keys(K, idx, S)
    assert K_T.shape[0] == 0
    np.testing.assert_allclose(orc.decode_attention(q, K_T, idx, K_r, V),
                               _dense_by_loops(q.tolist(), K.tolist(), V.tolist()), rtol=1e-12, atol=1e-13)


def test_pruning_zero_channels_changes_nothing():
    # channels that are identically zero on the prefix carry no logit mass:
    # pruning exactly those must reproduce dense attention
    rng = np.random.default_rng(12)
    S, D, R = 30, 10, 4
    q, K, V = rng.normal(size=D), rng.normal(size=(S, D)), rng.normal(size=(S, D))
    dead = [2, 5, 6]
    K[:S - R, dead] = 0.0
    Q_obs = rng.normal(size=(1, 4, D))
    score = orc.score_closed_form(Q_obs, np.where(np.arange(S)[:, None] < S - R, K, 0.0))
    idx = orc.select_top_T(score, D - len(dead))
    assert sorted(set(range(D)) - set(idx.tolist())) == dead
    K_T, K_r = orc.compact_keys(K, idx, R)
    np.testing.assert_allclose(orc.decode_attention(q, K_T, idx, K_r, V), orc.dense_attention(q, K, V),
                               rtol=1e-13, atol=1e-14)


def test_decode_output_is_a_convex_combination():
    rng = np.random.default_rng(13)
    S, D, R = 50, 8, 7
    q, K = rng.normal(size=D) * 4, rng.normal(size=(S, D))
    V = rng.normal(size=(S, D))
    idx = np.array([0, 3, 4, 6])
    K_T, K_r = orc.compact_keys(K, idx, R)
    out = orc.decode_attention(q, K_T, idx, K_r, V)
    assert (out <= V.max(0) + 1e-12).all() and (out >= V.min(0) - 1e-12).all()
    # constant values come back unchanged: the weights sum to one
    np.testing.assert_allclose(orc.decode_attention(q, K_T, idx, K_r, np.full((S, D), 2.5)), 2.5, rtol=1e-14)


def test_scale_uses_original_D():
    # one prefix token and one recent token with equal raw dot products but the
    # prefix one pruned to T = 1: logits are a/sqrt(D) with D = 4, not sqrt(T)
    D = 4
    a = 2.0
    q = np.array([a, 0.0, 0.0, 0.0])
    K_T = np.array([[1.0]])
    K_full = np.array([[0.0, 0.0, 0.0, 0.0]])
    V = np.array([[1.0, 0, 0, 0], [0.0, 0, 0, 0]])
    w = orc.decode_attention(q, K_T, np.array([0]), K_full, V)[0]
    assert abs(w - 1.0 / (1.0 + math.exp(-a / 2.0))) < 1e-15


def test_reprune_makes_recent_tokens_behave_like_prefix_tokens():
    # A cache built with S_recent = 64 whose 64 recent rows are then re-pruned must equal a cache built
    # with S_recent = 0 (the score uses all rows either way, so idx is the same); lambda = 0 stays dense.
    rng = np.random.default_rng(41)
    B, L, N_q, N_kv, D, S_obs, S = 1, 1, 4, 2, 16, 4, 200
    K = rng.normal(size=(B, S, L, N_kv, D)) * np.exp(rng.normal(size=D))
    V = rng.normal(size=(B, S, L, N_kv, D))
    Q = rng.normal(size=(B, S_obs, L, N_q, D))
    a = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, 64, 0.5)
    b = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, 0, 0.5)
    for o in (a, b):
        o.score_select(Q, K)
        o.compact(K, V)
    assert (a.idx == b.idx).all()
    a.reprune(keep_recent=0)
    for h in range(N_kv):
        assert (a.K_T[0][0][h] == b.K_T[0][0][h]).all() and a.K_full[0][0][h].shape[0] == 0
    k_new, v_new = rng.normal(size=(B, L, N_kv, D)), rng.normal(size=(B, L, N_kv, D))
    q = rng.normal(size=(B, L, N_q, D))
    for o in (a, b):
        o.append(k_new, v_new)
    np.testing.assert_allclose(a.decode_attn(q), b.decode_attn(q), rtol=1e-13, atol=1e-14)
    # keep_recent is honoured and only whole blocks move
    c = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, 100, 0.5)
    c.score_select(Q, K)
    c.compact(K, V)
    c.reprune(keep_recent=30)            # 100 - 30 = 70 movable -> one block of 64
    assert c.K_full[0][0][0].shape[0] == 36 and c.K_T[0][0][0].shape[0] == 100 + 64
    d = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, 100, 0.0)
    d.score_select(Q, K)
    d.compact(K, V)
    d.reprune(keep_recent=0)
    d.append(k_new, v_new)
    Kd = np.vstack([K[0, :, 0, 1], k_new[0, 0, 1][None]])
    Vd = np.vstack([V[0, :, 0, 1], v_new[0, 0, 1][None]])
    np.testing.assert_allclose(d.decode_attn(q)[0, 0, 2], _dense_by_loops(q[0, 0, 2].tolist(), Kd.tolist(), Vd.tolist()),
                               rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ behind a token-eviction method (Sec. 4.1)
def test_eviction_equals_masking_the_evicted_tokens():
    # Evicting a token from a head is the same as that token never receiving attention: with the evicted
    # key rows set to zero the literal Frobenius score is unchanged (zero rows add nothing), and dense
    # attention over the kept rows only must equal the path with lambda = 0 on the gathered tensors.
    rng = np.random.default_rng(77)
    B, L, N_q, N_kv, D, S_obs, S, n = 1, 2, 4, 2, 12, 3, 40, 17
    K = rng.normal(size=(B, S, L, N_kv, D)) * np.exp(rng.normal(size=D))
    V = rng.normal(size=(B, S, L, N_kv, D))
    Q = rng.normal(size=(B, S_obs, L, N_q, D))
    tok = np.zeros((B, L, N_kv, n), dtype=np.int64)
    for l in range(L):
        for h in range(N_kv):
            early = np.sort(rng.permutation(S - S_obs)[: n - S_obs])
            tok[0, l, h] = np.concatenate([early, np.arange(S - S_obs, S)])
    Kg, Vg = orc.gather_kept(K, tok, [n]), orc.gather_kept(V, tok, [n])
    assert Kg.shape == (B, n, L, N_kv, D)
    o = orc.ThinKOracle(B, L, N_q, N_kv, D, [n], S_obs, S_obs, 0.5)
    o.score_select(Q, Kg)
    for l in range(L):
        for h in range(N_kv):
            mask = np.zeros(S)
            mask[tok[0, l, h]] = 1.0
            Qg = np.stack([Q[0, :, l, h * 2 + g] for g in range(2)])
            want = orc.score_literal(Qg, K[0, :, l, h] * mask[:, None])
            np.testing.assert_allclose(o.score[0, l, h], want, rtol=1e-12)
            # different heads keep different tokens, and the gather follows each head's own list
            assert (Kg[0, :, l, h] == K[0, tok[0, l, h], l, h]).all()
    assert (tok[0, 0, 0] != tok[0, 0, 1]).any()
    d = orc.ThinKOracle(B, L, N_q, N_kv, D, [n], S_obs, S_obs, 0.0)
    d.score_select(Q, Kg)
    d.compact(Kg, Vg)
    q = rng.normal(size=(B, L, N_q, D))
    out = d.decode_attn(q)
    for l in range(L):
        for hq in range(N_q):
            h = hq // 2
            rows = tok[0, l, h].tolist()
            want = _dense_by_loops(q[0, l, hq].tolist(), K[0, rows, l, h].tolist(), V[0, rows, l, h].tolist())
            np.testing.assert_allclose(out[0, l, hq], want, rtol=1e-12, atol=1e-13)
    # identity list = no eviction
    ident = np.broadcast_to(np.arange(S), (B, L, N_kv, S))
    assert (orc.gather_kept(K, ident, [S]) == K).all()


# ------------------------------------------------------------------ value score (App. D)
def test_value_score_against_loops():
    rng = np.random.default_rng(21)
    G, S_obs, S, D = 2, 3, 9, 4
    Q, K, V = rng.normal(size=(G, S_obs, D)), rng.normal(size=(S, D)), rng.normal(size=(S, D))
    rows = [_dense_by_loops(Q[g, s].tolist(), K.tolist(), V.tolist()) for g in range(G) for s in range(S_obs)]
    want = [math.sqrt(sum(r[j] ** 2 for r in rows)) for j in range(D)]
    np.testing.assert_allclose(orc.score_value(Q, K, V), want, rtol=1e-12)


def test_value_score_uniform_attention_closed_form():
    # K = 0 makes every attention row uniform, so each output row is the column mean of V and the
    # score is sqrt(rows) * |mean_j|
    rng = np.random.default_rng(5)
    G, S_obs, S, D = 2, 3, 11, 6
    V = rng.normal(size=(S, D))
    got = orc.score_value(rng.normal(size=(G, S_obs, D)), np.zeros((S, D)), V)
    np.testing.assert_allclose(got, math.sqrt(G * S_obs) * np.abs(V.mean(axis=0)), rtol=1e-12)


def test_value_pruning_decode_equals_zeroed_prefix_channels():
    # ThinKV decode = ordinary ThinK decode on a value cache whose pruned channels are zero on the prefix
    # rows (computed by the other routine); lam_v = 0 is the ThinK path itself; a channel that is zero on
    # the prefix anyway can be pruned for free.
    rng = np.random.default_rng(9)
    B, L, N_q, N_kv, D, S_obs, S, R = 1, 1, 4, 2, 16, 4, 60, 8
    K = rng.normal(size=(B, S, L, N_kv, D)) * np.exp(rng.normal(size=D))
    V = rng.normal(size=(B, S, L, N_kv, D)) * np.exp(0.3 * rng.normal(size=D))
    Q = rng.normal(size=(B, S_obs, L, N_q, D))
    kv = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, R, 0.5, lam_v=0.25)
    kv.score_select(Q, K)
    kv.score_select_v(Q, K, V)
    assert kv.T_v == 12 and kv.idx_v.shape == (B, L, N_kv, 12)
    for h in range(N_kv):                      # selection = the ranked value scores of this head
        Qg = np.stack([Q[0, :, 0, h * 2 + g] for g in range(2)])
        s = orc.score_value(Qg, K[0, :, 0, h], V[0, :, 0, h])
        assert set(kv.idx_v[0, 0, h]) == set(np.argsort(-s, kind="stable")[:12])
        assert (np.diff(kv.idx_v[0, 0, h]) > 0).all()
    kv.compact(K, V)
    k_only = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, R, 0.5)
    k_only.score_select(Q, K)
    Vz = V.copy()
    for h in range(N_kv):
        dropped = np.setdiff1d(np.arange(D), kv.idx_v[0, 0, h])
        Vz[0, : S - R, 0, h][:, dropped] = 0.0
    k_only.compact(K, Vz)
    k_new, v_new = rng.normal(size=(B, L, N_kv, D)), rng.normal(size=(B, L, N_kv, D))
    q = rng.normal(size=(B, L, N_q, D))
    for o in (kv, k_only):
        o.append(k_new, v_new)
    np.testing.assert_allclose(kv.decode_attn(q), k_only.decode_attn(q), rtol=1e-12, atol=1e-14)
    # the tail (recent + new rows) kept its full values: the dropped channels of the output are not zero
    assert (np.abs(kv.decode_attn(q)) > 0).all()
    # lam_v = 0: nothing pruned
    full = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, R, 0.5, lam_v=0.0)
    full.score_select(Q, K)
    full.score_select_v(Q, K, V)
    assert (full.idx_v == np.arange(D)).all()
    full.compact(K, V)
    ref = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, R, 0.5)
    ref.score_select(Q, K)
    ref.compact(K, V)
    for o in (full, ref):
        o.append(k_new, v_new)
    np.testing.assert_allclose(full.decode_attn(q), ref.decode_attn(q), rtol=1e-12, atol=1e-14)
    # a channel that is zero on every row scores zero and is the first to go
    V0 = V.copy()
    V0[..., 5] = 0.0
    z = orc.ThinKOracle(B, L, N_q, N_kv, D, [S], S_obs, R, 0.5, lam_v=1.0 / 16)
    z.score_select(Q, K)
    z.score_select_v(Q, K, V0)
    assert all(5 not in z.idx_v[0, 0, h] for h in range(N_kv)) and z.T_v == 15


# ------------------------------------------------------------------ memory model
def test_sec31_example_13GB():
    (B, S, L, N, D, e, printed), = _rows("sec31_kv_example.txt")
    elems = orc.kv_cache_elements(int(B), int(S), int(L), int(N), int(D))
    assert elems == 2 * 13 * 2048 * 32 * 32 * 128
    assert round(elems * e / 2 ** 30) == printed       # 13.0 GiB


def test_table7_memory_column():
    # Mistral-7B-shaped accounting the table evidently uses: 32 layers x 32 heads x 128, fp16,
    # recent-size 32, kept fraction 1 - lambda = 0.6 (unfloored)
    L, N, D, e = 32, 32, 128, 2
    for kv, think_m, vanilla_m in _rows("table7_memory.txt"):
        kv = int(kv)
        m = orc.think_cache_elements([kv], L, N, D, keep=0.6, S_recent=32) * e / 2 ** 20
        assert round(m, 1) == think_m
        # the vanilla row is the KV-size whose full cache matches that memory
        kv_equal = math.ceil(m / (orc.kv_cache_elements(1, 1, L, N, D) * e / 2 ** 20))
        van = orc.kv_cache_elements(1, kv_equal, L, N, D) * e / 2 ** 20
        assert abs(van - vanilla_m) <= 0.05 + 1e-9
    # Sec. 4.3: KV-size 128 with ThinK(0.4) is matched by KV-size 109 without
    m128 = orc.think_cache_elements([128], L, N, D, keep=0.6, S_recent=32)
    assert math.ceil(m128 / orc.kv_cache_elements(1, 1, L, N, D)) == 109
    # a recent-size of 0 or 128 would NOT reproduce the column: the pin fixes S_recent = 32
    for R in (0, 128):
        assert round(orc.think_cache_elements([128], L, N, D, 0.6, R) * e / 2 ** 20, 1) != 54.4


def test_kv_saving_20_percent():
    (lam, printed), = _rows("sec41_kv_saving.txt")
    S = 10 ** 6       # long prompt: the recent rows vanish from the ratio
    dense = orc.kv_cache_elements(1, S, 1, 1, 128)
    thin = orc.think_cache_elements([S], 1, 1, 128, keep=1 - lam, S_recent=32)
    assert abs((1 - thin / dense) - printed) < 1e-4
    # with the floored integer T = 76 of D = 128 the saving is (128-76)/256
    thin_T = orc.think_cache_elements([S], 1, 1, 128, keep=orc.kept_channels(lam, 128) / 128, S_recent=32)
    assert abs((1 - thin_T / dense) - 52 / 256) < 1e-4


# ------------------------------------------------------------------ whole path
def test_path_on_tensors_matches_per_head_dense_when_lambda_zero():
    rng = np.random.default_rng(31)
    B, L, N_q, N_kv, D, S_obs, R = 2, 2, 4, 2, 8, 3, 2
    lens = [9, 6]
    K = rng.normal(size=(B, 9, L, N_kv, D))
    V = rng.normal(size=(B, 9, L, N_kv, D))
    Q = rng.normal(size=(B, S_obs, L, N_q, D))
    o = orc.ThinKOracle(B, L, N_q, N_kv, D, lens, S_obs, R, 0.0)
    o.score_select(Q, K)
    o.compact(K, V)
    k_new, v_new = rng.normal(size=(B, L, N_kv, D)), rng.normal(size=(B, L, N_kv, D))
    o.append(k_new, v_new)
    q = rng.normal(size=(B, L, N_q, D))
    out = o.decode_attn(q)
    for b in range(B):
        for l in range(L):
            for n in range(N_q):
                h = n // 2
                Kd = np.vstack([K[b, :lens[b], l, h], k_new[b, l, h][None]])
                Vd = np.vstack([V[b, :lens[b], l, h], v_new[b, l, h][None]])
                np.testing.assert_allclose(out[b, l, n], _dense_by_loops(q[b, l, n].tolist(), Kd.tolist(), Vd.tolist()),
                                           rtol=1e-12, atol=1e-13)


def test_path_literal_and_closed_scores_agree():
    rng = np.random.default_rng(32)
    B, L, N_q, N_kv, D, S_obs = 1, 1, 4, 2, 16, 4
    K = rng.normal(size=(B, 20, L, N_kv, D)) * np.exp(rng.normal(size=D))
    Q = rng.normal(size=(B, S_obs, L, N_q, D))
    a = orc.ThinKOracle(B, L, N_q, N_kv, D, [20], S_obs, 4, 0.5)
    b = orc.ThinKOracle(B, L, N_q, N_kv, D, [20], S_obs, 4, 0.5)
    ia = a.score_select(Q, K, literal=True)
    ib = b.score_select(Q, K, literal=False)
    assert (ia == ib).all()
    np.testing.assert_allclose(a.score, b.score, rtol=1e-12)
