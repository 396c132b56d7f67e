"""ctypes front end of the CPU oracle in ``ps_oracle.cpp`` (test infrastructure only).

Argument marshalling between numpy arrays and the C functions; no arithmetic of the
method lives here.  Weights and hidden states are handed over in their storage type:
``float32`` arrays for dtype 0, ``uint16`` arrays holding bf16 bit patterns for dtype 1.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ps_oracle.cpp")
_LIB = os.path.join(_HERE, "libps_oracle.so")

WEIGHT_NAMES = (
    "embed", "mask_embed", "mask_feat", "w_fc", "b_fc", "g_in", "w_q", "w_k", "w_v", "w_o",
    "g_post", "w_gate", "w_up", "w_down", "g_final", "w_lm",
)
TAP_NAMES = ("x_in", "x0", "xn", "q", "k_new", "v_new", "attn", "a", "an", "act", "hdn", "hn")


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, OpenMP over rows, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Config(C.Structure):
    _fields_ = [
        ("dtype", C.c_int), ("hidden", C.c_int), ("n_heads", C.c_int), ("n_kv_heads", C.c_int),
        ("head_dim", C.c_int), ("ffn", C.c_int), ("vocab", C.c_int), ("k_masks", C.c_int),
        ("max_batch", C.c_int), ("max_ctx", C.c_int), ("rope_base", C.c_double),
        ("rms_eps", C.c_double), ("has_fc_bias", C.c_int), ("no_fc", C.c_int),
    ]


class _Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES]


class _Taps(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in TAP_NAMES]


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build_oracle())
        _lib.pso_create.restype = C.c_void_p
        _lib.pso_create.argtypes = [C.POINTER(_Config), C.POINTER(_Weights)]
        _lib.pso_destroy.argtypes = [C.c_void_p]
        _lib.pso_kv_len.argtypes = [C.c_void_p, C.c_int]
        _lib.pso_kv_reset.argtypes = [C.c_void_p, C.c_int]
        _lib.pso_kv_import.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        _lib.pso_kv_export.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        _lib.pso_kv_append.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        _lib.pso_draft_step.argtypes = [
            C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
            C.POINTER(_Taps),
        ]
        _lib.pso_row_stats.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int] + [C.c_void_p] * 4
        _lib.pso_philox4x32.argtypes = [C.c_void_p] * 3
        _lib.pso_uniforms.argtypes = [
            C.c_uint64, C.c_uint64, C.c_int, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double),
        ]
        _lib.pso_verify.argtypes = (
            [C.c_int] * 4 + [C.c_void_p] * 3 + [C.c_double, C.c_uint64, C.c_uint64] + [C.c_void_p] * 7
        )
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


@dataclass
class OracleConfig:
    dtype: int
    hidden: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    k_masks: int
    max_batch: int
    max_ctx: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5
    no_fc: bool = False   # embedding-only input: no fc layer, no target feature


class Oracle:
    """One drafter (weights + per-slot KV caches) evaluated by the CPU oracle."""

    def __init__(self, cfg: OracleConfig, weights: dict):
        lib = _load()
        self.cfg = cfg
        self._np_dtype = np.float32 if cfg.dtype == 0 else np.uint16
        self._keep = {}
        w = _Weights()
        for name in WEIGHT_NAMES:
            arr = weights.get(name)
            if arr is None:
                setattr(w, name, None)
                continue
            arr = np.ascontiguousarray(arr)
            assert arr.dtype == self._np_dtype, (name, arr.dtype)
            self._keep[name] = arr
            setattr(w, name, arr.ctypes.data)
        c = _Config(
            cfg.dtype, cfg.hidden, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn, cfg.vocab,
            cfg.k_masks, cfg.max_batch, cfg.max_ctx, cfg.rope_base, cfg.rms_eps,
            1 if weights.get("b_fc") is not None else 0, 1 if cfg.no_fc else 0,
        )
        self._h = lib.pso_create(C.byref(c), C.byref(w))

    def __del__(self):
        if getattr(self, "_h", None):
            _load().pso_destroy(self._h)
            self._h = None

    def kv_len(self, slot: int) -> int:
        return _load().pso_kv_len(self._h, slot)

    def kv_reset(self, slot: int) -> None:
        _load().pso_kv_reset(self._h, slot)

    def kv_import(self, slot: int, K: np.ndarray, V: np.ndarray) -> None:
        K = np.ascontiguousarray(K, dtype=np.float64)
        V = np.ascontiguousarray(V, dtype=np.float64)
        rc = _load().pso_kv_import(self._h, slot, K.shape[0], _ptr(K), _ptr(V))
        assert rc == 0, rc

    def kv_export(self, slot: int):
        n = self.kv_len(slot)
        w = self.cfg.n_kv_heads * self.cfg.head_dim
        K = np.empty((n, w), np.float64)
        V = np.empty((n, w), np.float64)
        _load().pso_kv_export(self._h, slot, _ptr(K), _ptr(V))
        return K, V

    def kv_append(self, slot: int, hidden: np.ndarray, tokens: np.ndarray) -> int:
        hidden = np.ascontiguousarray(hidden)
        assert hidden.dtype == self._np_dtype
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        return _load().pso_kv_append(self._h, slot, len(tokens), _ptr(hidden), _ptr(tokens))

    def draft_step(self, slot: int, hidden_last: np.ndarray, token_last: int, k_use=None,
                   want_logits: bool = True, taps: bool = False):
        """Returns dict(logits [k+1][V], feat [k+1][H], and the taps if asked)."""
        cfg = self.cfg
        k_use = cfg.k_masks if k_use is None else k_use
        R = k_use + 1
        hidden_last = np.ascontiguousarray(hidden_last)
        assert hidden_last.dtype == self._np_dtype
        logits = np.empty((R, cfg.vocab), np.float64) if want_logits else None
        feat = np.empty((R, cfg.hidden), np.float64)
        out = {}
        t = None
        if taps:
            Hq = cfg.n_heads * cfg.head_dim
            Hkv = cfg.n_kv_heads * cfg.head_dim
            widths = dict(x_in=2 * cfg.hidden, x0=cfg.hidden, xn=cfg.hidden, q=Hq, k_new=Hkv,
                          v_new=Hkv, attn=Hq, a=cfg.hidden, an=cfg.hidden, act=cfg.ffn,
                          hdn=cfg.hidden, hn=cfg.hidden)
            t = _Taps()
            for n in TAP_NAMES:
                out[n] = np.empty((R, widths[n]), np.float64)
                setattr(t, n, out[n].ctypes.data)
        rc = _load().pso_draft_step(self._h, slot, _ptr(hidden_last), int(token_last), k_use,
                                    _ptr(logits), _ptr(feat), C.byref(t) if t is not None else None)
        if rc != 0:
            raise RuntimeError(f"oracle draft_step status {rc}")
        out["logits"] = logits
        out["feat"] = feat
        return out

    def group_forward(self, slot: int, hidden: np.ndarray, tokens: np.ndarray):
        """Group-wise parallel training layout, forward only (Sec. 4.1, Fig. 3): n groups of one
        real pair + k [MASK] rows.  Returns dict(logits [n][k+1][V], feat [n][k+1][H])."""
        cfg = self.cfg
        hidden = np.ascontiguousarray(hidden)
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        assert hidden.dtype == self._np_dtype and hidden.shape == (len(tokens), cfg.hidden)
        n, R = len(tokens), cfg.k_masks + 1
        logits = np.empty((n, R, cfg.vocab), np.float64)
        feat = np.empty((n, R, cfg.hidden), np.float64)
        lib = _load()
        lib.pso_group_forward.restype = C.c_int
        lib.pso_group_forward.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p]
        rc = lib.pso_group_forward(self._h, slot, n, _ptr(hidden), _ptr(tokens), _ptr(logits), _ptr(feat))
        if rc != 0:
            raise RuntimeError(f"oracle group_forward status {rc}")
        return dict(logits=logits, feat=feat)


def num_threads() -> int:
    """OpenMP threads the oracle's row loops run on."""
    return _load().pso_num_threads()


def set_threads(n: int) -> None:
    """Number of OpenMP threads the oracle's row loops use from now on."""
    _load().pso_set_threads(int(n))


def row_stats(logits: np.ndarray, top_n: int):
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    n, V = logits.shape
    row_max = np.empty(n, np.float64)
    row_lse = np.empty(n, np.float64)
    top_ids = np.empty((n, top_n), np.int32)
    top_logit = np.empty((n, top_n), np.float64)
    _load().pso_row_stats(_ptr(logits), n, V, top_n, _ptr(row_max), _ptr(row_lse), _ptr(top_ids),
                          _ptr(top_logit))
    return row_max, row_lse, top_ids, top_logit


def philox4x32(key, ctr) -> np.ndarray:
    key = np.ascontiguousarray(key, dtype=np.uint32)
    ctr = np.ascontiguousarray(ctr, dtype=np.uint32)
    out = np.empty(4, np.uint32)
    _load().pso_philox4x32(_ptr(key), _ptr(ctr), _ptr(out))
    return out


def uniforms(seed: int, offset: int, b: int, i: int):
    r = C.c_double()
    u2 = C.c_double()
    _load().pso_uniforms(seed, offset, b, i, C.byref(r), C.byref(u2))
    return r.value, u2.value


def verify(draft_tokens, draft_logits, target_logits, temperature: float, seed: int, offset: int):
    """Eq. 1 / Algorithm 1 (chain).  draft_tokens [B][n_draft], draft_logits [B][n_draft][V] or
    None, target_logits [B][n_target][V].  Returns a dict of numpy arrays."""
    draft_tokens = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    target_logits = np.ascontiguousarray(target_logits, dtype=np.float32)
    B, n_draft = draft_tokens.shape
    _, n_target, V = target_logits.shape
    if draft_logits is not None:
        draft_logits = np.ascontiguousarray(draft_logits, dtype=np.float32)
        assert draft_logits.shape == (B, n_draft, V)
    accept_len = np.empty(B, np.int32)
    out_tokens = np.empty((B, n_draft + 1), np.int32)
    n_out = np.empty(B, np.int32)
    margin_accept = np.empty((B, n_draft), np.float64)
    margin_cdf = np.empty(B, np.float64)
    nonfinite = np.empty(B, np.int32)
    neighbours = np.empty((B, 2), np.int32)
    rc = _load().pso_verify(B, n_draft, n_target, V, _ptr(draft_tokens), _ptr(draft_logits),
                            _ptr(target_logits), float(temperature), seed, offset, _ptr(accept_len),
                            _ptr(out_tokens), _ptr(n_out), _ptr(margin_accept), _ptr(margin_cdf),
                            _ptr(nonfinite), _ptr(neighbours))
    if rc != 0:
        raise ValueError(f"oracle verify status {rc}")
    return dict(accept_len=accept_len, out_tokens=out_tokens, n_out=n_out,
                margin_accept=margin_accept, margin_cdf=margin_cdf, nonfinite=nonfinite,
                neighbours=neighbours)


def verify_tree(parent, tokens, draft_logits, target_logits, temperature: float, seed: int, offset: int,
                max_depth: int | None = None):
    """Algorithm 1 in full.  parent [n_nodes] (-1: child of the root; children are tried in
    increasing node id), tokens [B][n_nodes], draft_logits [B][max_depth][V] (one row per tree
    depth) or None at temperature 0, target_logits [B][n_nodes+1][V] (row 0: after the prefix,
    row 1+i: after node i).  Returns a dict of numpy arrays."""
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    target_logits = np.ascontiguousarray(target_logits, dtype=np.float32)
    B, n_nodes = tokens.shape
    V = target_logits.shape[-1]
    assert target_logits.shape == (B, n_nodes + 1, V) and parent.shape == (n_nodes,)
    if draft_logits is not None:
        draft_logits = np.ascontiguousarray(draft_logits, dtype=np.float32)
        max_depth = draft_logits.shape[1] if max_depth is None else max_depth
        assert draft_logits.shape == (B, max_depth, V)
    assert max_depth is not None
    accept_len = np.empty(B, np.int32)
    out_tokens = np.empty((B, max_depth + 1), np.int32)
    n_out = np.empty(B, np.int32)
    path = np.empty((B, max_depth), np.int32)
    margin_accept = np.empty(B, np.float64)
    margin_cdf = np.empty(B, np.float64)
    nonfinite = np.empty(B, np.int32)
    lib = _load()
    lib.pso_verify_tree.restype = C.c_int
    lib.pso_verify_tree.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_void_p, C.c_double, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p,
                                    C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    neighbours = np.empty((B, 2), np.int32)
    rc = lib.pso_verify_tree(B, n_nodes, max_depth, V, _ptr(parent), _ptr(tokens), _ptr(draft_logits),
                             _ptr(target_logits), float(temperature), seed, offset, _ptr(accept_len),
                             _ptr(out_tokens), _ptr(n_out), _ptr(path), _ptr(margin_accept), _ptr(margin_cdf),
                             _ptr(nonfinite), _ptr(neighbours))
    if rc != 0:
        raise ValueError(f"oracle verify_tree status {rc}")
    return dict(accept_len=accept_len, out_tokens=out_tokens, n_out=n_out, path=path,
                margin_accept=margin_accept, margin_cdf=margin_cdf, nonfinite=nonfinite,
                neighbours=neighbours)


def build_tree(parent, rank, top_ids, sampled=None):
    """The draft tree of a static shape from per-depth top-n lists: parent, rank [n_nodes];
    top_ids [B][R][top_n] int32; sampled [B][R] int32 or None.  Returns tokens [B][n_nodes]."""
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    rank = np.ascontiguousarray(rank, dtype=np.int32)
    top_ids = np.ascontiguousarray(top_ids, dtype=np.int32)
    B, R, top_n = top_ids.shape
    if sampled is not None:
        sampled = np.ascontiguousarray(sampled, dtype=np.int32)
        assert sampled.shape == (B, R)
    tokens = np.empty((B, len(parent)), np.int32)
    lib = _load()
    lib.pso_build_tree.restype = C.c_int
    lib.pso_build_tree.argtypes = [C.c_int] * 4 + [C.c_void_p] * 5
    rc = lib.pso_build_tree(B, len(parent), R, top_n, _ptr(parent), _ptr(rank), _ptr(top_ids), _ptr(sampled),
                            _ptr(tokens))
    if rc != 0:
        raise ValueError(f"oracle build_tree status {rc}")
    return tokens


def gumbel_sample(logits, temperature: float, seed: int, offset: int, row_id):
    """One token per row from softmax(logits / T) by the Gumbel-max rule with the Philox stream
    of the draft sampler.  logits [rows][V] float64, row_id [rows] int (b | j << 8).
    Returns (tokens, margin): margin = best perturbed value minus the runner-up."""
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    row_id = np.ascontiguousarray(row_id, dtype=np.int32)
    n, V = logits.shape
    tokens = np.empty(n, np.int32)
    margin = np.empty(n, np.float64)
    lib = _load()
    lib.pso_gumbel_sample.restype = C.c_int
    lib.pso_gumbel_sample.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_double, C.c_uint64, C.c_uint64,
                                      C.c_void_p, C.c_void_p, C.c_void_p]
    rc = lib.pso_gumbel_sample(_ptr(logits), n, V, float(temperature), seed, offset, _ptr(row_id),
                               _ptr(tokens), _ptr(margin))
    if rc != 0:
        raise ValueError(f"oracle gumbel_sample status {rc}")
    return tokens, margin
