"""CPU oracle for ThinK (query-driven key-cache channel pruning).

TEST INFRASTRUCTURE.  Plain numpy in fp64, one head at a time, in the paper's
notation: Q_i, K_i, V_i in R^{S x D} for head i (Sec. 3.2).  Nothing here is
blocked, fused or reordered, and nothing here is used by the CUDA path (the two
share no code).  Only the tests, the smoke check and the benchmark's CPU
baseline call it.

What the paper fixes and what it leaves open
--------------------------------------------
* T = floor((1 - lambda) D) channels are kept per head (Sec. 3.1 below Eq. 1,
  and the trace constraint of Eq. 2).
* Score_i[j] = || Q_i[-S_obs:, j] K_i[:, j]^T ||_F (Sec. 3.2, "Observation
  Window"), all S key rows, no causal mask inside the window.
* I_i = Top_T(Score_i, T) (Sec. 3.2).  Ties: the lower channel index wins
  (declared reading; the paper does not say).  The kept set is stored ascending.
* Grouped-query attention: the G query heads that share a key head are stacked
  row-wise into one (G*S_obs) x D matrix before the norm is taken, i.e. the
  squared column norms are summed over the group (declared reading).
* The most recent S_recent prompt tokens and every newly decoded token keep all
  D key channels (Sec. 3.3); the pruned prefix keeps T.
* Decode (Sec. 3.3, Fig. 2): the query is pruned with the stored mask and
  multiplied with the pruned keys, the unpruned query with the unpruned keys;
  the two logit vectors are concatenated, scaled by 1/sqrt(D) with the
  original D, and go through ONE softmax; the value cache is untouched.

* Value-channel pruning (App. D): Score_v = column norms of the window's
  attention output, top-T_v kept.  App. D stops at the criterion; carrying it
  through decode like the keys (prefix rows thinned, recent and new rows whole,
  a pruned prefix channel counting as zero) is a declared reading.

Pins (tests/test_oracle_pins.py): rank-one Frobenius identity, Eq. 2's loss for
one pruned channel, brute-force subset search, lambda = 0 and S_recent = S
reducing to dense attention computed by a separately written routine, hand
computed softmax cases, and the memory figures the paper prints (Sec. 3.1
example, Table 7 "Memory(M)" column).  Unpinned by the paper (declared
readings only): the GQA aggregation and the tie rule -- "parity unpinned" for
those two choices.
"""
from __future__ import annotations

import math
from typing import List, Sequence

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Sec. 3.1 / Eq. 2: number of kept channels
# --------------------------------------------------------------------------
def kept_channels(lam: float, D: int) -> int:
    """T = floor((1 - lambda) D).  A 1e-9 guard keeps products such as
    (1 - 0.4) * 5 = 2.9999999999999996 from flooring one too low."""
    if not (0.0 <= lam < 1.0):
        raise ValueError("lambda must be in [0, 1)")
    T = int(math.floor((1.0 - lam) * D + 1e-9))
    if T < 1:
        raise ValueError("T must be >= 1")
    return T


# --------------------------------------------------------------------------
# Sec. 3.2: channel score, literal definition
# --------------------------------------------------------------------------
def score_literal(Q_obs: np.ndarray, K: np.ndarray) -> np.ndarray:
    """Score[j] = || Q[-S_obs:, j] K[:, j]^T ||_F, formed as the matrix it is.

    Q_obs: [G, S_obs, D] window rows of the G query heads of the group
           (G = 1 for multi-head attention), K: [S, D].
    """
    Q_obs = np.asarray(Q_obs, dtype=F64)
    K = np.asarray(K, dtype=F64)
    G, S_obs, D = Q_obs.shape
    stacked = Q_obs.reshape(G * S_obs, D)
    score = np.empty(D, dtype=F64)
    for j in range(D):
        M = np.outer(stacked[:, j], K[:, j])       # (G*S_obs) x S interaction matrix
        score[j] = math.sqrt(float(np.sum(M * M)))
    return score


def score_closed_form(Q_obs: np.ndarray, K: np.ndarray) -> np.ndarray:
    """The same quantity through || a b^T ||_F = ||a||_2 ||b||_2."""
    Q_obs = np.asarray(Q_obs, dtype=F64)
    K = np.asarray(K, dtype=F64)
    qn2 = np.sum(Q_obs * Q_obs, axis=(0, 1))
    kn2 = np.sum(K * K, axis=0)
    return np.sqrt(qn2 * kn2)


# --------------------------------------------------------------------------
# Sec. 3.1 Eq. 1: magnitude-based criterion (the paper's own baseline)
# --------------------------------------------------------------------------
def score_magnitude(K: np.ndarray, p: int) -> np.ndarray:
    """M[d] = || K[:, d] ||_p for p in {1, 2} (Eq. 1)."""
    K = np.asarray(K, dtype=F64)
    if p == 1:
        return np.sum(np.abs(K), axis=0)
    if p == 2:
        return np.sqrt(np.sum(K * K, axis=0))
    raise ValueError("p must be 1 or 2")


# --------------------------------------------------------------------------
# Sec. 3.2: I_i = Top_T(Score_i, T)
# --------------------------------------------------------------------------
def select_top_T(score: np.ndarray, T: int) -> np.ndarray:
    """Indices of the T largest scores; equal scores go to the lower index;
    returned ascending (a mask written as a list)."""
    score = np.asarray(score, dtype=F64)
    D = score.shape[0]
    order = sorted(range(D), key=lambda j: (-score[j], j))
    return np.array(sorted(order[:T]), dtype=np.int64)


def near_tie(score: np.ndarray, T: int, rel: float = 1e-6) -> bool:
    """True when the T-th and (T+1)-th largest scores differ by less than
    ``rel`` relative: the cut is then decided by rounding."""
    s = np.sort(np.asarray(score, dtype=F64))[::-1]
    if T >= s.shape[0]:
        return False
    a, b = s[T - 1], s[T]
    return (a - b) <= rel * max(abs(a), abs(b))


# --------------------------------------------------------------------------
# Eq. 2: the objective the greedy rule stands in for (diagnostic)
# --------------------------------------------------------------------------
def pruning_loss(Q: np.ndarray, K: np.ndarray, keep: Sequence[int]) -> float:
    """|| Q K^T - Q S K^T ||_F with S = diag(1 on kept channels) (Eq. 2)."""
    Q = np.asarray(Q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    s = np.zeros(Q.shape[1], dtype=F64)
    s[list(keep)] = 1.0
    full = Q @ K.T
    pruned = (Q * s[None, :]) @ K.T
    return float(np.linalg.norm(full - pruned, "fro"))


# --------------------------------------------------------------------------
# Sec. 3.3: two-part key cache
# --------------------------------------------------------------------------
def compact_keys(K: np.ndarray, idx: np.ndarray, S_recent: int):
    """Split K [S, D] into the pruned prefix K_T [S - S_recent, T] (kept
    channels only, in ascending channel order) and the unpruned recent rows
    [S_recent, D]."""
    K = np.asarray(K)
    S = K.shape[0]
    S_p = S - S_recent
    return K[:S_p][:, idx].copy(), K[S_p:].copy()


# --------------------------------------------------------------------------
# Sec. 3.2 attention and Sec. 3.3 decode over the two-part cache
# --------------------------------------------------------------------------
def _softmax(x: np.ndarray) -> np.ndarray:
    e = np.exp(x - np.max(x))
    return e / np.sum(e)


def decode_attention(q: np.ndarray, K_T: np.ndarray, idx: np.ndarray, K_full: np.ndarray,
                     V: np.ndarray) -> np.ndarray:
    """One query row against the two-part cache of its key head.

    q: [D]; K_T: [S_p, T] pruned keys; idx: [T] kept channels; K_full: [U, D]
    unpruned keys (recent prompt rows followed by decoded tokens); V: [S_p + U,
    D] all value rows in token order.  Returns [D].
    """
    q = np.asarray(q, dtype=F64)
    D = q.shape[0]
    q_T = q[idx]                                           # query pruned by the mask
    x_p = np.asarray(K_T, dtype=F64) @ q_T                 # pruned query x pruned keys
    x_r = np.asarray(K_full, dtype=F64) @ q                # unpruned query x unpruned keys
    x = np.concatenate([x_p, x_r]) / math.sqrt(D)          # concatenated; sqrt of the ORIGINAL D
    p = _softmax(x)
    return p @ np.asarray(V, dtype=F64)


def dense_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """softmax(q K^T / sqrt(D)) V for one query row (Sec. 3.2)."""
    q = np.asarray(q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    V = np.asarray(V, dtype=F64)
    x = (K @ q) / math.sqrt(q.shape[0])
    return _softmax(x) @ V


# --------------------------------------------------------------------------
# App. D Eqs. 3-4: value-channel score
# --------------------------------------------------------------------------
def score_value(Q_obs: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """Score_v[j] = || softmax(Q[-S_obs:] K^T / sqrt(D)) V[:, j] ||_F, with the
    group's query heads stacked row-wise as for the key score."""
    Q_obs = np.asarray(Q_obs, dtype=F64)
    K = np.asarray(K, dtype=F64)
    V = np.asarray(V, dtype=F64)
    G, S_obs, D = Q_obs.shape
    Qs = Q_obs.reshape(G * S_obs, D)
    X = (Qs @ K.T) / math.sqrt(D)
    X = X - X.max(axis=1, keepdims=True)
    P = np.exp(X)
    P /= P.sum(axis=1, keepdims=True)
    O = P @ V                                             # (G*S_obs) x D
    return np.sqrt(np.sum(O * O, axis=0))


def decode_attention_kv(q: np.ndarray, K_T: np.ndarray, idx: np.ndarray, K_full: np.ndarray, V_T: np.ndarray,
                        idx_v: np.ndarray, V_full: np.ndarray) -> np.ndarray:
    """App. D carried through decode the way Sec. 3.3 treats the keys (declared reading: App. D gives
    the criterion only): the values of the pruned prefix keep T_v channels, V_T [S_p, T_v] with kept
    channels idx_v; recent and decoded tokens keep full rows, V_full [U, D].  The attention weights are
    those of decode_attention; a pruned value channel of a prefix token counts as zero, so the output
    channel j sums the tail's share everywhere and the prefix's share only where j is kept."""
    q = np.asarray(q, dtype=F64)
    D = q.shape[0]
    x_p = np.asarray(K_T, dtype=F64) @ q[idx]
    x_r = np.asarray(K_full, dtype=F64) @ q
    p = _softmax(np.concatenate([x_p, x_r]) / math.sqrt(D))
    S_p = x_p.shape[0]
    out = p[S_p:] @ np.asarray(V_full, dtype=F64)
    out[idx_v] += p[:S_p] @ np.asarray(V_T, dtype=F64)
    return out


# --------------------------------------------------------------------------
# Sec. 3.1 cache-size model and the Table 7 accounting
# --------------------------------------------------------------------------
def kv_cache_elements(B: int, S: int, L: int, N: int, D: int) -> int:
    """2 x B x S x L x N x D (Sec. 3.1)."""
    return 2 * B * S * L * N * D


def think_cache_elements(seq_lens: Sequence[int], L: int, N: int, D: int, keep: float, S_recent: int,
                         new_tokens: int = 0) -> float:
    """Elements held by the two-part cache: pruned prefix keys at ``keep`` x D
    channels, unpruned recent + decoded keys at D, all values at D (Sec. 3.3).
    ``keep`` is the kept fraction of channels (T / D for an integer T; the
    paper's Table 7 figures correspond to keep = 1 - lambda unfloored)."""
    total = 0.0
    for S in seq_lens:
        S_p = S - S_recent
        k = S_p * keep * D + (S_recent + new_tokens) * D
        v = (S + new_tokens) * D
        total += (k + v) * L * N
    return total


# --------------------------------------------------------------------------
# Sec. 4.1: ThinK behind a token-eviction method (H2O, SnapKV): that method
# first reduces every head to "KV-size" tokens; ThinK then prunes the channels
# of the keys that survived.  The eviction method itself is an input here (a
# list of kept tokens per head); this routine only forms the compressed tensors
# that the method would hand over.
# --------------------------------------------------------------------------
def gather_kept(X: np.ndarray, tok: np.ndarray, kept: Sequence[int]) -> np.ndarray:
    """X [B, S, L, N, D], tok [B, L, N, >= kept[b]] (rows of X), kept[b] tokens per head
    -> [B, max kept, L, N, D] with out[b, i, l, h] = X[b, tok[b, l, h, i], l, h]; rows past
    kept[b] are NaN (never to be read)."""
    B, _, L, N, D = X.shape
    out = np.full((B, max(kept), L, N, D), np.nan, dtype=F64)
    for b in range(B):
        for l in range(L):
            for h in range(N):
                for i in range(kept[b]):
                    out[b, i, l, h] = X[b, tok[b, l, h, i], l, h]
    return out


# --------------------------------------------------------------------------
# The whole path on the paper's B x S x L x N x D tensors, step by step
# --------------------------------------------------------------------------
class ThinKOracle:
    """Runs prefill scoring/selection/compaction and the decode steps for every
    (batch entry, layer, key head), with the per-head routines above."""

    def __init__(self, B: int, L: int, N_q: int, N_kv: int, D: int, seq_lens: Sequence[int], S_obs: int,
                 S_recent: int, lam: float, lam_v: float = 0.0):
        assert N_q % N_kv == 0
        self.B, self.L, self.N_q, self.N_kv, self.D = B, L, N_q, N_kv, D
        self.G = N_q // N_kv
        self.seq_lens = [int(s) for s in seq_lens]
        self.S_obs, self.S_recent, self.lam = S_obs, S_recent, lam
        self.T = kept_channels(lam, D)
        self.idx = None
        self.score = None
        # App. D: value channels are pruned too when lam_v > 0
        self.lam_v = lam_v
        self.T_v = kept_channels(lam_v, D)
        self.idx_v = None
        self.score_v = None

    # prefill, steps 1-3
    def score_select(self, Q_obs: np.ndarray, K: np.ndarray, literal: bool = False):
        """Q_obs [B, S_obs, L, N_q, D], K [B, S_max, L, N_kv, D] (float64)."""
        B, L, N_kv, D, G = self.B, self.L, self.N_kv, self.D, self.G
        self.idx = np.zeros((B, L, N_kv, self.T), dtype=np.int64)
        self.score = np.zeros((B, L, N_kv, D), dtype=F64)
        fn = score_literal if literal else score_closed_form
        for b in range(B):
            S_b = self.seq_lens[b]
            for l in range(L):
                for h in range(N_kv):
                    Qg = np.stack([Q_obs[b, :, l, h * G + g, :] for g in range(G)])   # [G, S_obs, D]
                    s = fn(Qg, K[b, :S_b, l, h, :])
                    self.score[b, l, h] = s
                    self.idx[b, l, h] = select_top_T(s, self.T)
        return self.idx

    # App. D Eqs. 3-4: value-channel scores and their top-T_v
    def score_select_v(self, Q_obs: np.ndarray, K: np.ndarray, V: np.ndarray):
        B, L, N_kv, D, G = self.B, self.L, self.N_kv, self.D, self.G
        self.idx_v = np.zeros((B, L, N_kv, self.T_v), dtype=np.int64)
        self.score_v = np.zeros((B, L, N_kv, D), dtype=F64)
        for b in range(B):
            S_b = self.seq_lens[b]
            for l in range(L):
                for h in range(N_kv):
                    Qg = np.stack([Q_obs[b, :, l, h * G + g, :] for g in range(G)])
                    s = score_value(Qg, K[b, :S_b, l, h, :], V[b, :S_b, l, h, :])
                    self.score_v[b, l, h] = s
                    self.idx_v[b, l, h] = select_top_T(s, self.T_v)
        return self.idx_v

    # prefill, step 4
    def compact(self, K: np.ndarray, V: np.ndarray):
        B, L, N_kv = self.B, self.L, self.N_kv
        self.K_T = [[[None] * N_kv for _ in range(L)] for _ in range(B)]
        self.K_full = [[[None] * N_kv for _ in range(L)] for _ in range(B)]
        self.V_all = [[[None] * N_kv for _ in range(L)] for _ in range(B)]
        for b in range(B):
            S_b = self.seq_lens[b]
            for l in range(L):
                for h in range(N_kv):
                    kt, kr = compact_keys(np.asarray(K[b, :S_b, l, h, :], dtype=F64), self.idx[b, l, h],
                                          self.S_recent)
                    self.K_T[b][l][h] = kt
                    self.K_full[b][l][h] = kr
                    self.V_all[b][l][h] = np.array(V[b, :S_b, l, h, :], dtype=F64)
        if self.idx_v is not None:
            # the prefix values keep their T_v channels, recent rows stay whole (same split as the keys)
            self.V_T = [[[None] * N_kv for _ in range(L)] for _ in range(B)]
            for b in range(B):
                S_p = self.seq_lens[b] - self.S_recent
                for l in range(L):
                    for h in range(N_kv):
                        va = self.V_all[b][l][h]
                        self.V_T[b][l][h] = va[:S_p][:, self.idx_v[b, l, h]].copy()
                        self.V_all[b][l][h] = va[S_p:].copy()       # from here on: the unpruned value rows only

    # decode, step 5
    def append(self, k_new: np.ndarray, v_new: np.ndarray):
        """k_new, v_new [B, L, N_kv, D]: the new token's key stays unpruned."""
        for b in range(self.B):
            for l in range(self.L):
                for h in range(self.N_kv):
                    self.K_full[b][l][h] = np.vstack([self.K_full[b][l][h], np.asarray(k_new[b, l, h], F64)[None]])
                    self.V_all[b][l][h] = np.vstack([self.V_all[b][l][h], np.asarray(v_new[b, l, h], F64)[None]])

    # App. C.1 control flow without the quantiser: prune the oldest unpruned keys, join them to K_T
    def reprune(self, keep_recent: int, block: int = 64):
        """Moves whole blocks of `block` tokens, oldest first, from the unpruned keys to the pruned
        ones (kept channels only, the idx selected at prefill) while >= keep_recent stay unpruned."""
        for b in range(self.B):
            for l in range(self.L):
                for h in range(self.N_kv):
                    n = self.K_full[b][l][h].shape[0]
                    m = max(0, (n - keep_recent) // block) * block
                    if m == 0:
                        continue
                    moved = self.K_full[b][l][h][:m][:, self.idx[b, l, h]]
                    self.K_T[b][l][h] = np.vstack([self.K_T[b][l][h], moved])
                    self.K_full[b][l][h] = self.K_full[b][l][h][m:]

    # decode, steps 6-9
    def decode_attn(self, q: np.ndarray) -> np.ndarray:
        """q [B, L, N_q, D] -> out [B, L, N_q, D]."""
        out = np.zeros((self.B, self.L, self.N_q, self.D), dtype=F64)
        for b in range(self.B):
            for l in range(self.L):
                for h in range(self.N_kv):
                    for g in range(self.G):
                        n = h * self.G + g
                        if self.idx_v is None:
                            out[b, l, n] = decode_attention(q[b, l, n], self.K_T[b][l][h], self.idx[b, l, h],
                                                            self.K_full[b][l][h], self.V_all[b][l][h])
                        else:
                            out[b, l, n] = decode_attention_kv(q[b, l, n], self.K_T[b][l][h], self.idx[b, l, h],
                                                               self.K_full[b][l][h], self.V_T[b][l][h],
                                                               self.idx_v[b, l, h], self.V_all[b][l][h])
        return out
