"""Seeded synthetic workloads: post-RoPE Q/K/V activations shaped like the
paper's LLaMA / Mistral runs (Sec. 4.1 "Implementation Details").

This module only draws inputs.  It holds none of the method's arithmetic
(no scores, no selection, no attention) and is the one module that both the
CUDA path's callers and the CPU oracle's tests import.

Key/query law.  The paper observes (Sec. 3, Fig. 4) that a few key channels
carry much larger magnitudes than the rest across all tokens while values show
no such pattern.  The generator reproduces that structure: every (layer, head,
channel) draws a standard deviation sigma ~ LogNormal(0, 1), optionally a few
random "outlier" channels per head are multiplied by a constant, and every
token draws N(0, sigma^2) in that channel.  Queries follow the same law with
independent draws.  Values are N(0, 1).  Where a config asks for RoPE the
rotation acts on channel pairs (j, j + D/2) with angle pos * theta^(-2j/D);
rounding to the storage type happens after the rotation.
"""
from __future__ import annotations

import dataclasses
import functools
from typing import List, Optional, Tuple

import torch

__all__ = ["Workload", "CONFIGS", "get_config", "shrink", "make_prefill", "make_step", "make_eviction", "evicted"]


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                 # "bf16" | "f32"
    B: int
    L: int
    N_q: int
    N_kv: int
    D: int
    seq_lens: Tuple[int, ...]  # one per batch entry
    S_obs: int
    lam: float                 # pruning ratio lambda
    steps: int                 # decode steps
    rope_theta: Optional[float]
    outliers: Optional[Tuple[int, float]]  # (channels per head, factor)
    seed: int
    S_recent: Optional[int] = None         # default: S_obs

    @property
    def S_max(self) -> int:
        return max(self.seq_lens)

    @property
    def recent(self) -> int:
        return self.S_obs if self.S_recent is None else self.S_recent

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4


def _ragged(seed: int, B: int, lo: int, hi: int) -> Tuple[int, ...]:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return tuple(int(x) for x in torch.randint(lo, hi + 1, (B,), generator=g))


CONFIGS = {
    # tiny single layer, fp32, MHA
    "c1": Workload("c1", "f32", 1, 1, 4, 4, 64, (512,), 32, 0.5, 8, None, (4, 10.0), 0x74170001),
    # LLaMA-3-8B-shaped
    "c2": Workload("c2", "bf16", 1, 32, 32, 8, 128, (8192,), 32, 0.4, 64, 500000.0, None, 0x74170002),
    # Mistral-7B-shaped, batch of 4 long prompts
    "c3": Workload("c3", "bf16", 4, 32, 32, 8, 128, (32768,) * 4, 32, 0.5, 128, 1.0e6, None, 0x74170003),
    # LLaMA-2-7B-shaped MHA batch-throughput case, ragged
    "c4": Workload("c4", "bf16", 16, 32, 32, 32, 128, _ragged(0x74170004, 16, 2048, 4096), 32, 0.6, 256,
                   None, (8, 20.0), 0x74170004),
    # long-context stress
    "c5": Workload("c5", "bf16", 1, 32, 32, 8, 128, (131072,), 64, 0.5, 512, 500000.0, None, 0x74170005),
}


def get_config(name: str) -> Workload:
    return CONFIGS[name]


def shrink(w: Workload, *, S: Optional[int] = None, L: Optional[int] = None, B: Optional[int] = None,
           steps: Optional[int] = None, lam: Optional[float] = None, name: Optional[str] = None) -> Workload:
    """Same head geometry and law, smaller extent (for parity tests)."""
    B2 = w.B if B is None else B
    lens = [w.seq_lens[i % len(w.seq_lens)] for i in range(B2)]
    if S is not None:
        longest = max(lens)
        # keep the ragged profile: scale every length, never below the window
        lens = [max(w.S_obs + 1, (x * S + longest - 1) // longest) for x in lens]
    return dataclasses.replace(
        w, name=name or (w.name + "-small"), B=B2, L=w.L if L is None else L, seq_lens=tuple(lens),
        steps=w.steps if steps is None else steps, lam=w.lam if lam is None else lam)


def evicted(w: Workload, kv_sizes) -> Workload:
    """The workload a cache sees behind a token-eviction method that kept kv_sizes[b] tokens per head."""
    if isinstance(kv_sizes, int):
        kv_sizes = (kv_sizes,) * w.B
    assert len(kv_sizes) == w.B and all(w.recent <= n <= s and w.S_obs <= n for n, s in zip(kv_sizes, w.seq_lens))
    return dataclasses.replace(w, name=w.name + "-evicted", seq_lens=tuple(int(n) for n in kv_sizes))


def make_eviction(w: Workload, kv_sizes, device="cpu") -> torch.Tensor:
    """Stand-in for the output of an upstream token-eviction method (H2O / SnapKV style): for every
    (b, l, h) the observation window (last S_obs prompt rows) plus a seeded random subset of the earlier
    rows, kv_sizes[b] rows in all, ascending.  int32 [B, L, N_kv, max kv_size]; unused slots hold -1."""
    if isinstance(kv_sizes, int):
        kv_sizes = (kv_sizes,) * w.B
    width = max(kv_sizes)
    tok = torch.full((w.B, w.L, w.N_kv, width), -1, dtype=torch.int32)
    for b in range(w.B):
        S_b, n = w.seq_lens[b], int(kv_sizes[b])
        assert w.S_obs <= n <= S_b
        early = S_b - w.S_obs
        key = torch.rand((w.L, w.N_kv, max(early, 1)), generator=_gen("cpu", w.seed, 9, b))
        pick = torch.topk(key, n - w.S_obs, dim=-1).indices.sort(dim=-1).values if n > w.S_obs else \
            torch.empty((w.L, w.N_kv, 0), dtype=torch.int64)
        window = torch.arange(early, S_b).expand(w.L, w.N_kv, w.S_obs)
        tok[b, :, :, :n] = torch.cat([pick, window], dim=-1).to(torch.int32)
    return tok.to(device)


def _gen(device, seed: int, *ids: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = seed & 0xFFFFFFFF
    for i in ids:
        s = (s * 0x9E3779B1 + (i + 1) * 0x85EBCA6B + 0x27D4EB2F) & 0x7FFFFFFFFFFFFFFF
    g.manual_seed(s)
    return g


@functools.lru_cache(maxsize=16)
def _sigma_cpu(w: Workload, tensor_id: int, n_heads: int) -> torch.Tensor:
    g = _gen("cpu", w.seed, 100 + tensor_id)
    sig = torch.exp(torch.randn((w.L, n_heads, w.D), generator=g, dtype=torch.float32))
    if w.outliers is not None:
        n_out, factor = w.outliers
        for l in range(w.L):
            for h in range(n_heads):
                ch = torch.randperm(w.D, generator=g)[:n_out]
                sig[l, h, ch] *= factor
    return sig


def _sigma(w: Workload, tensor_id: int, n_heads: int, device) -> torch.Tensor:
    """Per (layer, head, channel) standard deviation, float32 [L, n_heads, D]."""
    return _sigma_cpu(w, tensor_id, n_heads).to(device)


def _rope(x: torch.Tensor, pos: torch.Tensor, theta: float) -> torch.Tensor:
    """x [..., S, N, D] float32, pos [S] (token positions); rotates pairs (j, j+D/2)."""
    D = x.shape[-1]
    half = D // 2
    j = torch.arange(half, device=x.device, dtype=torch.float64)
    inv = torch.pow(torch.tensor(theta, dtype=torch.float64, device=x.device), -2.0 * j / D)
    ang = pos.to(torch.float64)[:, None] * inv[None, :]          # [S, half]
    cos = torch.cos(ang).to(torch.float32)[:, None, :]
    sin = torch.sin(ang).to(torch.float32)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return torch.cat([a * cos - b * sin, a * sin + b * cos], dim=-1)


TENSOR_K, TENSOR_V, TENSOR_Q = 1, 2, 3


def _draw(w: Workload, tensor_id: int, sig_l: Optional[torch.Tensor], n_heads: int, b: int, l: int,
          pos: torch.Tensor, device, step_tag: int = 0) -> torch.Tensor:
    """One (batch entry, layer) slab [len(pos), n_heads, D] in float32, before rounding."""
    g = _gen(device, w.seed, tensor_id, b, l, step_tag)
    x = torch.randn((pos.numel(), n_heads, w.D), generator=g, device=device, dtype=torch.float32)
    if sig_l is not None:
        x = x * sig_l[None, :, :]
        if w.rope_theta is not None:
            x = _rope(x, pos, w.rope_theta)
    return x


def make_prefill(w: Workload, device="cpu", pad_nan: bool = True):
    """Prompt tensors in the paper's B x S x L x N x D layout (Sec. 1).

    Returns dict with K, V [B, S_max, L, N_kv, D], Q_obs [B, S_obs, L, N_q, D]
    (the last S_obs query rows of every sequence) and seq_lens.  Rows at or
    beyond a sequence's length hold NaN when ``pad_nan`` so that any read of
    them shows up in the results.
    """
    dt = w.torch_dtype
    fill = float("nan") if pad_nan else 0.0
    K = torch.full((w.B, w.S_max, w.L, w.N_kv, w.D), fill, dtype=dt, device=device)
    V = torch.full((w.B, w.S_max, w.L, w.N_kv, w.D), fill, dtype=dt, device=device)
    Q = torch.empty((w.B, w.S_obs, w.L, w.N_q, w.D), dtype=dt, device=device)
    sig_k = _sigma(w, TENSOR_K, w.N_kv, device)
    sig_q = _sigma(w, TENSOR_Q, w.N_q, device)
    for b in range(w.B):
        Sb = w.seq_lens[b]
        pos = torch.arange(Sb, device=device)
        for l in range(w.L):
            K[b, :Sb, l] = _draw(w, TENSOR_K, sig_k[l], w.N_kv, b, l, pos, device).to(dt)
            V[b, :Sb, l] = _draw(w, TENSOR_V, None, w.N_kv, b, l, pos, device).to(dt)
            Q[b, :, l] = _draw(w, TENSOR_Q, sig_q[l], w.N_q, b, l, pos[Sb - w.S_obs:], device).to(dt)
    return {"K": K, "V": V, "Q_obs": Q, "seq_lens": list(w.seq_lens)}


def make_step(w: Workload, t: int, device="cpu"):
    """Inputs of decode step t: q [B, L, N_q, D], k_new, v_new [B, L, N_kv, D]
    for the token at position S_b + t of every sequence."""
    dt = w.torch_dtype
    q = torch.empty((w.B, w.L, w.N_q, w.D), dtype=dt, device=device)
    k = torch.empty((w.B, w.L, w.N_kv, w.D), dtype=dt, device=device)
    v = torch.empty((w.B, w.L, w.N_kv, w.D), dtype=dt, device=device)
    sig_k = _sigma(w, TENSOR_K, w.N_kv, device)
    sig_q = _sigma(w, TENSOR_Q, w.N_q, device)
    for b in range(w.B):
        pos = torch.tensor([w.seq_lens[b] + t], device=device)
        for l in range(w.L):
            q[b, l] = _draw(w, TENSOR_Q, sig_q[l], w.N_q, b, l, pos, device, 1 + t)[0].to(dt)
            k[b, l] = _draw(w, TENSOR_K, sig_k[l], w.N_kv, b, l, pos, device, 1 + t)[0].to(dt)
            v[b, l] = _draw(w, TENSOR_V, None, w.N_kv, b, l, pos, device, 1 + t)[0].to(dt)
    return {"q": q, "k_new": k, "v_new": v}
