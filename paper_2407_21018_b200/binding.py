"""ctypes binding of libthink.so -- argument marshalling only.

Every step of the path runs in the library's CUDA kernels; this module turns
torch tensors into pointers/strides, allocates the caller-owned buffers with
``torch.empty`` and forwards the current CUDA stream.  Importing it raises if
the compiled library is missing: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libthink.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} not found: build it first (python -m paper_2407_21018_b200.build); "
        "the CUDA library is the only implementation of this path")

lib = C.CDLL(LIB_PATH)

THINK_OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_STATE, ERR_CAPACITY, ERR_CUDA = range(6)
BF16, F32 = 0, 1
SCORE_QUERY_DRIVEN, SCORE_KEY_L2, SCORE_KEY_L1 = 0, 1, 2
VALUE_SCORE_AUTO, VALUE_SCORE_MMA_SYNC = 0, 1
ERR_BIT_TOKEN_RANGE, ERR_BIT_WAIT_TIMEOUT, ERR_BIT_SMEM_ALIGN, ERR_BIT_NON_FINITE = 1, 2, 4, 8
TILE_TOKENS = 64


class Config(C.Structure):
    _fields_ = [("B", C.c_int32), ("L", C.c_int32), ("N_q", C.c_int32), ("N_kv", C.c_int32), ("D", C.c_int32),
                ("S_max", C.c_int32), ("S_obs", C.c_int32), ("S_recent", C.c_int32),
                ("max_new_tokens", C.c_int32), ("dtype", C.c_int32), ("criterion", C.c_int32),
                ("value_score_kernel", C.c_int32), ("lam", C.c_double), ("lam_v", C.c_double)]


class Tensor5(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("stride_b", C.c_int64), ("stride_s", C.c_int64),
                ("stride_l", C.c_int64), ("stride_n", C.c_int64)]


class Sizes(C.Structure):
    _fields_ = [("k_thin", C.c_size_t), ("tail_k", C.c_size_t), ("tail_v", C.c_size_t), ("idx", C.c_size_t),
                ("scores", C.c_size_t), ("workspace", C.c_size_t), ("model_think_bytes", C.c_size_t),
                ("model_dense_bytes", C.c_size_t), ("v_thin", C.c_size_t), ("perm_v", C.c_size_t)]


EXPORTS = {
    "thinK_T": (C.c_int32, [C.c_double, C.c_int32]),
    "thinK_status_string": (C.c_char_p, [C.c_int]),
    "thinK_cache_bytes": (C.c_int, [C.POINTER(Config), C.POINTER(C.c_int32), C.POINTER(Sizes)]),
    "thinK_create": (C.c_int, [C.POINTER(Config), C.POINTER(C.c_int32), C.POINTER(Sizes)] + [C.c_void_p] * 6 +
                     [C.POINTER(C.c_void_p)]),
    "thinK_score_select": (C.c_int, [C.c_void_p, Tensor5, Tensor5, C.c_int32, C.c_int32, C.c_void_p]),
    "thinK_compact": (C.c_int, [C.c_void_p, Tensor5, Tensor5, C.c_int32, C.c_int32, C.c_void_p]),
    "thinK_prefill": (C.c_int, [C.c_void_p, Tensor5, Tensor5, Tensor5, C.c_int32, C.c_int32, C.c_void_p]),
    "thinK_attach_value_cache": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "thinK_score_select_kv": (C.c_int, [C.c_void_p, Tensor5, Tensor5, Tensor5, C.c_int32, C.c_int32, C.c_void_p]),
    "thinK_prefill_evicted": (C.c_int, [C.c_void_p, Tensor5, Tensor5, Tensor5, C.c_void_p, C.c_int64, C.c_int32,
                                        C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "thinK_v_kept_bytes": (C.c_size_t, [C.c_void_p]),
    "thinK_append": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "thinK_append_decode": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                      C.c_void_p]),
    "thinK_decode_attn": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "thinK_score_select_static": (C.c_int, [C.POINTER(Config), C.POINTER(C.c_int32), Tensor5, Tensor5, C.c_int32,
                                            C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "thinK_reprune_tail": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
    "thinK_repruned_len": (C.c_int32, [C.c_void_p, C.c_int32]),
    "thinK_tail_len": (C.c_int32, [C.c_void_p, C.c_int32]),
    "thinK_device_error": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32)]),
    "thinK_destroy": (C.c_int, [C.c_void_p]),
}
for _name, (_res, _args) in EXPORTS.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class ThinKError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.thinK_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != THINK_OK:
        raise ThinKError(status, where)


def thinK_T(lam: float, D: int) -> int:
    return int(lib.thinK_T(lam, D))


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.bfloat16:
        return BF16
    if dt == torch.float32:
        return F32
    raise ThinKError(ERR_UNSUPPORTED, "dtype")


def tensor5(t: Optional[torch.Tensor]) -> Tensor5:
    """View of a 5-d tensor indexed [b, s, l, n, d] with d contiguous (any strides otherwise)."""
    if t is None:
        return Tensor5(None, 0, 0, 0, 0)
    assert t.dim() == 5 and t.stride(4) == 1
    return Tensor5(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2), t.stride(3))


def make_config(B, L, N_q, N_kv, D, S_max, S_obs, S_recent, max_new_tokens, lam, dtype, criterion=SCORE_QUERY_DRIVEN,
                lam_v=0.0, value_score_kernel=VALUE_SCORE_AUTO):
    return Config(B, L, N_q, N_kv, D, S_max, S_obs, S_recent, max_new_tokens,
                  dtype if isinstance(dtype, int) else _dtype_code(dtype), criterion, value_score_kernel, float(lam),
                  float(lam_v))


def thinK_cache_bytes(cfg: Config, seq_lens: Sequence[int]) -> Sizes:
    arr = (C.c_int32 * len(seq_lens))(*seq_lens)
    out = Sizes()
    _check(lib.thinK_cache_bytes(C.byref(cfg), arr, C.byref(out)), "thinK_cache_bytes")
    return out


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def score_select_static(cfg: Config, seq_lens: Sequence[int], q_obs: Optional[torch.Tensor], k: torch.Tensor,
                        idx: torch.Tensor, scores: Optional[torch.Tensor] = None, layer0=0, nlayers=None, stream=None):
    """thinK_score_select_static: same results as ThinKCache.score_select, but the library brings its
    own fixed scratch, so nothing is allocated by the call (for callers that may not allocate device
    memory).  `idx` (uint8) and `scores` (float64, optional) are caller-provided outputs."""
    nlayers = cfg.L - layer0 if nlayers is None else nlayers
    arr = (C.c_int32 * len(seq_lens))(*seq_lens)
    _check(lib.thinK_score_select_static(C.byref(cfg), arr, tensor5(q_obs), tensor5(k), layer0, nlayers,
                                         idx.data_ptr(), scores.data_ptr() if scores is not None else None,
                                         _stream_ptr(stream)), "thinK_score_select_static")


class ThinKCache:
    """Owns the caller-side buffers (torch allocations) and the library handle."""

    def __init__(self, cfg: Config, seq_lens: Sequence[int], device="cuda", keep_scores: bool = True):
        self.cfg = cfg
        self.seq_lens = [int(s) for s in seq_lens]
        self.sizes = thinK_cache_bytes(cfg, self.seq_lens)
        self.device = torch.device(device)
        self.T = thinK_T(cfg.lam, cfg.D)
        self.torch_dtype = torch.bfloat16 if cfg.dtype == BF16 else torch.float32
        self.elem = 2 if cfg.dtype == BF16 else 4
        mk = lambda n: torch.empty(max(int(n), 256), dtype=torch.uint8, device=self.device)
        self.k_thin = mk(self.sizes.k_thin)
        self.tail_k = mk(self.sizes.tail_k)
        self.tail_v = mk(self.sizes.tail_v)
        self.idx = mk(self.sizes.idx)
        self.scores = mk(self.sizes.scores) if keep_scores else None
        self.workspace = mk(self.sizes.workspace)
        self._v = None
        arr = (C.c_int32 * len(self.seq_lens))(*self.seq_lens)
        h = C.c_void_p()
        # what was actually allocated, for the library's own size check
        have = Sizes(self.k_thin.numel(), self.tail_k.numel(), self.tail_v.numel(), self.idx.numel(),
                     self.scores.numel() if self.scores is not None else 0, self.workspace.numel(), 0, 0,
                     max(int(self.sizes.v_thin), 256) if cfg.lam_v > 0 else 0,
                     max(int(self.sizes.perm_v), 256) if cfg.lam_v > 0 else 0)
        with torch.cuda.device(self.device):
            _check(lib.thinK_create(C.byref(cfg), arr, C.byref(have), self.k_thin.data_ptr(), self.tail_k.data_ptr(),
                                    self.tail_v.data_ptr(), self.idx.data_ptr(),
                                    self.scores.data_ptr() if self.scores is not None else None,
                                    self.workspace.data_ptr(), C.byref(h)), "thinK_create")
        self.handle = h
        self.T_v = thinK_T(cfg.lam_v, cfg.D)
        self.v_thin = self.perm_v = None
        if cfg.lam_v > 0:                      # value-channel pruning: two more caller-owned buffers
            self.v_thin, self.perm_v = mk(self.sizes.v_thin), mk(self.sizes.perm_v)
            self.scores_v = mk(self.sizes.scores) if keep_scores else None
            _check(lib.thinK_attach_value_cache(self.handle, self.v_thin.data_ptr(), self.perm_v.data_ptr(),
                                                self.scores_v.data_ptr() if self.scores_v is not None else None),
                   "thinK_attach_value_cache")

    def score_select_kv(self, q_obs: torch.Tensor, k: torch.Tensor, v: torch.Tensor, layer0=0, nlayers=None, stream=None):
        """Key scores + value scores (App. D) and both selections."""
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        _check(lib.thinK_score_select_kv(self.handle, tensor5(q_obs), tensor5(k), tensor5(v), layer0, nlayers,
                                         _stream_ptr(stream)), "thinK_score_select_kv")

    def scores_v_tensor(self) -> torch.Tensor:
        c = self.cfg
        return self.scores_v[: c.B * c.L * c.N_kv * c.D * 8].view(torch.float64).view(c.B, c.L, c.N_kv, c.D)

    def perm_v_tensor(self) -> torch.Tensor:
        """uint8 [B, L, N_kv, D]: kept value channels ascending ([..., :T_v]), then the pruned ones."""
        c = self.cfg
        return self.perm_v[: c.B * c.L * c.N_kv * c.D].view(c.B, c.L, c.N_kv, c.D)

    # -- the four calls of the path -------------------------------------
    def score_select(self, q_obs: Optional[torch.Tensor], k: torch.Tensor, layer0=0, nlayers=None, stream=None):
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        _check(lib.thinK_score_select(self.handle, tensor5(q_obs), tensor5(k), layer0, nlayers, _stream_ptr(stream)),
               "thinK_score_select")

    def compact(self, k: torch.Tensor, v: torch.Tensor, layer0=0, nlayers=None, stream=None):
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        self._v = v   # borrowed by the library: keep it alive
        _check(lib.thinK_compact(self.handle, tensor5(k), tensor5(v), layer0, nlayers, _stream_ptr(stream)),
               "thinK_compact")

    def prefill(self, q_obs: Optional[torch.Tensor], k: torch.Tensor, v: torch.Tensor, layer0=0, nlayers=None,
                stream=None):
        """score_select + compact in one call."""
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        self._v = v   # borrowed by the library: keep it alive
        _check(lib.thinK_prefill(self.handle, tensor5(q_obs), tensor5(k), tensor5(v), layer0, nlayers,
                                 _stream_ptr(stream)), "thinK_prefill")

    def prefill_evicted(self, q_obs: Optional[torch.Tensor], k: torch.Tensor, v: torch.Tensor, tok: torch.Tensor,
                        layer0=0, nlayers=None, stream=None):
        """Prefill behind a token-eviction method: tok int32 [B, L, N_kv, >= n_b] lists each head's kept rows of
        k and v (this cache was created with seq_lens = kept counts)."""
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        assert tok.dtype == torch.int32 and tok.dim() == 4 and tok.is_contiguous() and tok.is_cuda
        assert tuple(tok.shape[:3]) == (self.cfg.B, self.cfg.L, self.cfg.N_kv)
        if self._v is None:
            self._v = torch.empty(max(int(lib.thinK_v_kept_bytes(self.handle)), 256), dtype=torch.uint8,
                                  device=self.device)
        _check(lib.thinK_prefill_evicted(self.handle, tensor5(q_obs), tensor5(k), tensor5(v), tok.data_ptr(),
                                         tok.shape[3], k.shape[1], self._v.data_ptr(), layer0, nlayers,
                                         _stream_ptr(stream)), "thinK_prefill_evicted")

    def append(self, k_new: torch.Tensor, v_new: torch.Tensor, layer0=0, nlayers=None, stream=None):
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        assert k_new.is_contiguous() and v_new.is_contiguous()
        _check(lib.thinK_append(self.handle, k_new.data_ptr(), v_new.data_ptr(), layer0, nlayers, _stream_ptr(stream)),
               "thinK_append")

    def decode_attn(self, q: torch.Tensor, out: Optional[torch.Tensor] = None, layer0=0, nlayers=None, stream=None):
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        assert q.is_contiguous()
        if out is None:
            out = torch.empty_like(q)
        _check(lib.thinK_decode_attn(self.handle, q.data_ptr(), out.data_ptr(), layer0, nlayers, _stream_ptr(stream)),
               "thinK_decode_attn")
        return out

    def append_decode(self, k_new: torch.Tensor, v_new: torch.Tensor, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                      layer0=0, nlayers=None, stream=None):
        """append + decode_attn in one call (the attention kernel overlaps the append)."""
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        assert k_new.is_contiguous() and v_new.is_contiguous() and q.is_contiguous()
        if out is None:
            out = torch.empty_like(q)
        _check(lib.thinK_append_decode(self.handle, k_new.data_ptr(), v_new.data_ptr(), q.data_ptr(), out.data_ptr(),
                                       layer0, nlayers, _stream_ptr(stream)), "thinK_append_decode")
        return out

    def reprune_tail(self, keep_recent: int, layer0=0, nlayers=None, stream=None):
        """Thins the oldest whole 64-token blocks of the unpruned tail, keeping >= keep_recent unpruned."""
        nlayers = self.cfg.L - layer0 if nlayers is None else nlayers
        _check(lib.thinK_reprune_tail(self.handle, keep_recent, layer0, nlayers, _stream_ptr(stream)),
               "thinK_reprune_tail")

    def repruned_len(self, layer=0) -> int:
        return int(lib.thinK_repruned_len(self.handle, layer))

    # -- inspection ------------------------------------------------------
    def tail_len(self, layer=0) -> int:
        return int(lib.thinK_tail_len(self.handle, layer))

    def device_error(self) -> int:
        code = C.c_int32(0)
        _check(lib.thinK_device_error(self.handle, C.byref(code)), "thinK_device_error")
        return code.value

    def idx_tensor(self) -> torch.Tensor:
        c = self.cfg
        n = c.B * c.L * c.N_kv * self.T
        return self.idx[:n].view(c.B, c.L, c.N_kv, self.T)

    def scores_tensor(self) -> torch.Tensor:
        c = self.cfg
        n = c.B * c.L * c.N_kv * c.D * 8
        return self.scores[:n].view(torch.float64).view(c.B, c.L, c.N_kv, c.D)

    def close(self):
        if getattr(self, "handle", None):
            lib.thinK_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---------------------------------------------------------------------------
# Address arithmetic of the documented library layouts (for readers of k_thin /
# tail_k, e.g. tests): pure indexing, no arithmetic of the method.
# ---------------------------------------------------------------------------
def padded_T(T: int, dtype_code: int) -> int:
    """Rows stored per thin tile: bf16 pads T to a multiple of 8."""
    return (T + 7) & ~7 if dtype_code == BF16 else T


def _offsets_f32(rows: int, device) -> torch.Tensor:
    """Element offset of (row c, token u) in a channel-major swizzled fp32 tile [rows][64]."""
    c = torch.arange(rows, device=device)[:, None]
    u = torch.arange(TILE_TOKENS, device=device)[None, :]
    byte = u * 4
    return c * TILE_TOKENS + ((((byte >> 4) ^ (c & 7)) << 4) | (byte & 15)) // 4


def _offsets_bf16(Cp: int, device) -> torch.Tensor:
    """Element offset of (channel c, token u) in a bf16 tile of 64 tokens x Cp channels stored in
    MMA-fragment order (see include/think.h)."""
    c = torch.arange(Cp, device=device)[:, None]
    u = torch.arange(TILE_TOKENS, device=device)[None, :]
    n16 = Cp >> 4
    step, jx, r = u >> 4, (u >> 3) & 1, u & 7
    base = step * Cp * 32
    s, w = c >> 4, c & 15
    half, q, lo = w >> 3, (w & 7) >> 1, w & 1
    main = base + s * 512 + (r * 4 + q) * 16 + (jx * 2 + half) * 4 + lo * 2
    w8 = c - n16 * 16
    q8, lo8 = w8 >> 1, w8 & 1
    tail8 = base + n16 * 512 + (r * 4 + q8) * 8 + jx * 4 + lo8 * 2
    return torch.where(c < n16 * 16, main, tail8) // 2


def unpack_tiles(raw: torch.Tensor, n_tiles: int, rows: int, n_tokens: int) -> torch.Tensor:
    """raw: flat tensor (bf16 or fp32) holding n_tiles key tiles of `rows` channels x 64 tokens in
    the library layout of its dtype; returns the logical [n_tokens, rows] matrix."""
    t = raw[: n_tiles * rows * TILE_TOKENS].view(n_tiles, rows * TILE_TOKENS)
    off = _offsets_bf16(rows, raw.device) if raw.dtype == torch.bfloat16 else _offsets_f32(rows, raw.device)
    logical = t[:, off.reshape(-1)].view(n_tiles, rows, TILE_TOKENS)           # [tile, channel, u]
    return logical.permute(0, 2, 1).reshape(n_tiles * TILE_TOKENS, rows)[:n_tokens]


def k_thin_logical(cache: ThinKCache, b: int, l: int, h: int) -> torch.Tensor:
    """Pruned keys of one head as [S_p + re-pruned tokens, T]."""
    c = cache.cfg
    S_p = cache.seq_lens[b] - c.S_recent
    nt = [(s - c.S_recent + TILE_TOKENS - 1) // TILE_TOKENS for s in cache.seq_lens]
    cap = max(1, c.S_recent + c.max_new_tokens)
    re_cap = (cap + TILE_TOKENS - 1) // TILE_TOKENS      # tiles reserved per head for re-pruned tail blocks
    base = sum(c.L * c.N_kv * (x + re_cap) for x in nt[:b]) + (l * c.N_kv + h) * (nt[b] + re_cap)
    flat = cache.k_thin.view(cache.torch_dtype)
    Tp = padded_T(cache.T, c.dtype)
    per = Tp * TILE_TOKENS
    full = unpack_tiles(flat[base * per:(base + nt[b]) * per], nt[b], Tp, S_p)
    n_re = cache.repruned_len(l) // TILE_TOKENS            # re-pruned tail blocks follow the prompt's tiles
    if n_re:
        more = unpack_tiles(flat[(base + nt[b]) * per:(base + nt[b] + n_re) * per], n_re, Tp, n_re * TILE_TOKENS)
        full = torch.cat([full, more], dim=0)
    assert Tp == cache.T or not full[:, cache.T:].any(), "padding rows of a thin tile must be zero"
    return full[:, :cache.T]


def tail_logical(cache: ThinKCache, b: int, l: int, h: int):
    """Unpruned tail of one head: (keys [n, D], values [n, D]), re-pruned blocks excluded."""
    c = cache.cfg
    n = cache.tail_len(l)
    cap = max(1, c.S_recent + c.max_new_tokens)
    ttc = (cap + TILE_TOKENS - 1) // TILE_TOKENS
    unit = (b * c.L + l) * c.N_kv + h
    per = c.D * TILE_TOKENS
    flat = cache.tail_k.view(cache.torch_dtype)
    m = cache.repruned_len(l)                              # these tokens now live in k_thin
    keys = unpack_tiles(flat[unit * ttc * per:(unit + 1) * ttc * per], ttc, c.D, n)[m:]
    vals = cache.tail_v.view(cache.torch_dtype)[unit * cap * c.D:(unit * cap + n) * c.D].view(n, c.D)[m:]
    if cache.perm_v is not None:                           # stored in the permuted channel order: undo it
        perm = cache.perm_v_tensor()[b, l, h].long()
        out = torch.empty_like(vals)
        out[:, perm] = vals
        vals = out
    return keys, vals


def v_thin_logical(cache: ThinKCache, b: int, l: int, h: int) -> torch.Tensor:
    """Thinned prefix values of one head, [S_p, T_v] (kept channels ascending)."""
    c = cache.cfg
    Tvp = (cache.T_v + 15) // 16 * 16
    base = sum(c.L * c.N_kv * (cache.seq_lens[bb] - c.S_recent) * Tvp for bb in range(b))
    S_p = cache.seq_lens[b] - c.S_recent
    off = base + (l * c.N_kv + h) * S_p * Tvp
    rows = cache.v_thin.view(cache.torch_dtype)[off: off + S_p * Tvp].view(S_p, Tvp)
    assert (rows[:, cache.T_v:] == 0).all(), "padding channels of v_thin must be zero"
    return rows[:, : cache.T_v]
