"""Thin ctypes binding of the C ABI in include/ps.h.

Argument marshalling only: torch tensors supply device memory and the CUDA stream; every
step of the path runs in the library's kernels.  There is no CPU fallback: if the shared
library is missing or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

PS_OK = 0
STATUS_NAMES = {0: "PS_OK", -1: "PS_ERR_INVALID_ARG", -2: "PS_ERR_UNSUPPORTED", -3: "PS_ERR_CAPACITY",
                -4: "PS_ERR_CUDA", -5: "PS_ERR_TIMEOUT", -6: "PS_ERR_NONFINITE"}
PS_DTYPE_F32, PS_DTYPE_BF16 = 0, 1
PS_FLAG_FC_BIAS, PS_FLAG_UNFUSED_KERNELS, PS_FLAG_MMA_SYNC_GEMM, PS_FLAG_NO_FC = 1, 2, 4, 8
PS_FLAG_STAGE_LAUNCHES = 16
PS_MAX_BATCH, PS_MAX_MASKS, PS_MAX_TOP_N = 128, 15, 8

WEIGHT_NAMES = (
    "embed", "mask_embed", "mask_feat", "w_fc", "b_fc", "g_in", "w_q", "w_k", "w_v", "w_o",
    "g_post", "w_gate", "w_up", "w_down", "g_final", "w_lm",
)

EXPORTS = (
    "ps_workspace_bytes", "ps_init", "ps_kv_append", "ps_draft_step", "ps_verify", "ps_round_host",
    "ps_kv_len", "ps_kv_reset", "ps_kv_export", "ps_kv_import", "ps_poll", "ps_launch_count",
    "ps_last_error", "ps_destroy", "ps_philox_fill", "ps_profile", "ps_profile_read",
    "ps_verify_static", "ps_debug_buffer", "ps_verify_tree", "ps_draft_step_sampled", "ps_group_forward",
    "ps_build_tree", "ps_debug_wait_expires", "ps_debug_check_guards",
)


class PsError(RuntimeError):
    def __init__(self, status: int, text: str = ""):
        self.status = status
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {text}")


class ps_config(C.Structure):
    _fields_ = [
        ("dtype", C.c_int), ("hidden", C.c_int), ("n_heads", C.c_int), ("n_kv_heads", C.c_int),
        ("head_dim", C.c_int), ("ffn", C.c_int), ("vocab", C.c_int), ("k_masks", C.c_int),
        ("max_batch", C.c_int), ("max_ctx", C.c_int), ("rope_base", C.c_float),
        ("rms_eps", C.c_float), ("flags", C.c_int),
    ]


class ps_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES]


_lib = None


def load_library(path: str | None = None) -> C.CDLL:
    """Loads libps_b200.so (building it with nvcc if the in-tree copy is stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = path or _build.build()
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path}: the CUDA library is not built")
    lib = C.CDLL(path)
    vp, ip = C.c_void_p, C.POINTER(C.c_int)
    lib.ps_workspace_bytes.restype = C.c_size_t
    lib.ps_workspace_bytes.argtypes = [C.POINTER(ps_config)]
    lib.ps_init.argtypes = [C.POINTER(vp), C.POINTER(ps_config), C.POINTER(ps_weights), vp, C.c_size_t, vp]
    lib.ps_kv_append.argtypes = [vp, C.c_int, ip, ip, ip, vp, vp, vp]
    lib.ps_draft_step.argtypes = [vp, C.c_int, ip, vp, vp, C.c_int, vp, vp, vp, vp, vp, vp, vp]
    lib.ps_verify.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, vp, vp, C.c_float, C.c_uint64,
                              C.c_uint64, vp, vp, vp, vp]
    lib.ps_round_host.argtypes = [vp, C.c_int, ip, vp, vp, vp, C.c_float, C.c_uint64, C.c_uint64,
                                  vp, vp, vp, vp]
    lib.ps_draft_step_sampled.argtypes = [vp, C.c_int, ip, vp, vp, C.c_float, C.c_uint64, C.c_uint64, vp,
                                          C.c_int, vp, vp, vp, vp, vp, vp, vp]
    lib.ps_group_forward.argtypes = [vp, C.c_int, C.c_int, vp, vp, C.c_int, vp, vp, vp, vp, vp, vp, vp]
    lib.ps_verify_tree.argtypes = [vp, C.c_int, C.c_int, ip, vp, vp, vp, C.c_float, C.c_uint64, C.c_uint64,
                                   vp, vp, vp, vp, vp]
    lib.ps_build_tree.argtypes = [vp, C.c_int, C.c_int, ip, ip, vp, C.c_int, vp, vp, vp]
    lib.ps_debug_wait_expires.argtypes = [vp, C.c_longlong, vp]
    lib.ps_debug_check_guards.argtypes = [vp, vp, ip]
    lib.ps_kv_len.argtypes = [vp, C.c_int, ip]
    lib.ps_kv_reset.argtypes = [vp, C.c_int]
    lib.ps_kv_export.argtypes = [vp, C.c_int, vp, vp, vp]
    lib.ps_kv_import.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp]
    lib.ps_poll.argtypes = [vp, vp]
    lib.ps_launch_count.restype = C.c_longlong
    lib.ps_launch_count.argtypes = [vp]
    lib.ps_last_error.restype = C.c_char_p
    lib.ps_last_error.argtypes = [vp]
    lib.ps_destroy.restype = None
    lib.ps_destroy.argtypes = [vp]
    lib.ps_philox_fill.argtypes = [C.POINTER(C.c_uint32), vp, vp, C.c_int, vp]
    lib.ps_profile.argtypes = [vp, C.c_int]
    lib.ps_profile_read.argtypes = [vp, C.c_int, C.c_char_p, C.POINTER(C.c_float), ip, ip]
    lib.ps_debug_buffer.argtypes = [vp, C.c_char_p, C.POINTER(vp), C.POINTER(C.c_size_t)]
    lib.ps_verify_static.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp, C.c_float,
                                     C.c_uint64, C.c_uint64, vp, vp, vp, vp, C.c_char_p, C.c_size_t, vp]
    _lib = lib
    return lib


def _dptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _iarr(xs):
    return (C.c_int * len(xs))(*[int(x) for x in xs])


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def workspace_bytes(cfg: ps_config) -> int:
    return load_library().ps_workspace_bytes(C.byref(cfg))


def philox_fill(key, ctr: torch.Tensor) -> torch.Tensor:
    """out[i] = Philox-4x32-10(key, ctr[i]); ctr: CUDA int32/uint32 tensor [n][4]."""
    lib = load_library()
    out = torch.empty_like(ctr)
    k = (C.c_uint32 * 2)(int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF)
    rc = lib.ps_philox_fill(k, _dptr(ctr), _dptr(out), ctr.shape[0], _stream())
    if rc != PS_OK:
        raise PsError(rc)
    return out


def verify_static(draft_tokens: torch.Tensor, draft_logits, target_logits: torch.Tensor,
                  temperature: float, seed: int, offset: int, out: dict, nonfinite_flag=None,
                  stream=None) -> dict:
    """ps_verify_static: the acceptance test for callers that may not allocate device memory.

    Needs no Drafter and no workspace; the kernel's scratch is a fixed array inside the library
    (one per GPU, shared by all calls, so calls must not overlap on a GPU).  ``out`` must hold the
    caller's preallocated CUDA int32 tensors ``accept_len`` [B], ``out_tokens`` [B][n_draft+1] and
    ``n_out`` [B]: this wrapper allocates nothing either.
    """
    lib = load_library()
    B, n_draft = draft_tokens.shape
    _, n_target, vocab = target_logits.shape
    err = C.create_string_buffer(256)
    rc = lib.ps_verify_static(vocab, B, n_draft, n_target, _dptr(draft_tokens), _dptr(draft_logits),
                              _dptr(target_logits), float(temperature), seed, offset,
                              _dptr(out["accept_len"]), _dptr(out["out_tokens"]), _dptr(out["n_out"]),
                              _dptr(nonfinite_flag), err, 256, _stream(stream))
    if rc != PS_OK:
        raise PsError(rc, err.value.decode())
    return out


class Drafter:
    """One ps_ctx: a drafter with its KV caches on the current CUDA device.

    ``weights`` maps the names of ps_weights to CUDA tensors (float32 for dtype 0, bfloat16
    for dtype 1); the workspace is a torch uint8 tensor owned by this object.
    """

    def __init__(self, *, dtype: int, hidden: int, n_heads: int, n_kv_heads: int, head_dim: int,
                 ffn: int, vocab: int, k_masks: int, max_batch: int, max_ctx: int,
                 weights: dict, rope_base: float = 10000.0, rms_eps: float = 1e-5, flags: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2410_05589_b200 needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        if weights.get("b_fc") is not None:
            flags |= PS_FLAG_FC_BIAS
        self.cfg = ps_config(dtype, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab, k_masks,
                             max_batch, max_ctx, rope_base, rms_eps, flags)
        self.torch_dtype = torch.float32 if dtype == PS_DTYPE_F32 else torch.bfloat16
        self.weights = {}
        w = ps_weights()
        for n in WEIGHT_NAMES:
            t = weights.get(n)
            if t is not None:
                assert t.dtype == self.torch_dtype and t.is_cuda, n
                t = t.contiguous()
                self.weights[n] = t
                setattr(w, n, t.data_ptr())
        nbytes = self.lib.ps_workspace_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise PsError(-2, "configuration rejected by ps_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        h = C.c_void_p()
        rc = self.lib.ps_init(C.byref(h), C.byref(self.cfg), C.byref(w), _dptr(self.workspace),
                              nbytes, _stream())
        if rc != PS_OK:
            raise PsError(rc, "ps_init")
        self.h = h
        self.rows = k_masks + 1

    def close(self):
        if getattr(self, "h", None):
            self.lib.ps_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def _check(self, rc):
        if rc != PS_OK:
            raise PsError(rc, (self.lib.ps_last_error(self.h) or b"").decode())

    # ---- cache -------------------------------------------------------------------------
    def kv_len(self, slot: int) -> int:
        n = C.c_int()
        self._check(self.lib.ps_kv_len(self.h, slot, C.byref(n)))
        return n.value

    def kv_reset(self, slot: int) -> None:
        self._check(self.lib.ps_kv_reset(self.h, slot))

    def kv_append(self, seq_slot, n_new, hidden: torch.Tensor, tokens: torch.Tensor, stream=None):
        off = [0]
        for n in n_new:
            off.append(off[-1] + int(n))
        self._check(self.lib.ps_kv_append(self.h, len(seq_slot), _iarr(seq_slot), _iarr(n_new),
                                          _iarr(off), _dptr(hidden), _dptr(tokens), _stream(stream)))

    def kv_export(self, slot: int):
        n = self.kv_len(slot)
        w = self.cfg.n_kv_heads * self.cfg.head_dim
        K = torch.empty((n, w), dtype=self.torch_dtype, device="cuda")
        V = torch.empty_like(K)
        self._check(self.lib.ps_kv_export(self.h, slot, _dptr(K), _dptr(V), _stream()))
        return K, V

    def kv_import(self, slot: int, K: torch.Tensor, V: torch.Tensor):
        self._check(self.lib.ps_kv_import(self.h, slot, K.shape[0], _dptr(K), _dptr(V), _stream()))

    # ---- the hot path ------------------------------------------------------------------
    def draft_step(self, seq_slot, hidden_last: torch.Tensor, token_last: torch.Tensor, top_n: int = 1,
                   want_logits: bool = True, want_feat: bool = False, out: dict | None = None,
                   stream=None) -> dict:
        """ps_draft_step.  ``out`` may carry preallocated output tensors to reuse."""
        B, R, V, H = len(seq_slot), self.rows, self.cfg.vocab, self.cfg.hidden
        o = out if out is not None else {}
        dev = "cuda"
        if "row_max" not in o:
            o["top_ids"] = torch.empty((B, R, max(top_n, 1)), dtype=torch.int32, device=dev)
            o["top_logit"] = torch.empty((B, R, max(top_n, 1)), dtype=torch.float32, device=dev)
            o["row_max"] = torch.empty((B, R), dtype=torch.float32, device=dev)
            o["row_lse"] = torch.empty((B, R), dtype=torch.float32, device=dev)
            o["logits"] = torch.empty((B, R, V), dtype=torch.float32, device=dev) if want_logits else None
            o["feat"] = torch.empty((B, R, H), dtype=torch.float32, device=dev) if want_feat else None
        self._check(self.lib.ps_draft_step(
            self.h, B, _iarr(seq_slot), _dptr(hidden_last), _dptr(token_last), top_n,
            _dptr(o["top_ids"]), _dptr(o["top_logit"]), _dptr(o["row_max"]), _dptr(o["row_lse"]),
            _dptr(o.get("logits")), _dptr(o.get("feat")), _stream(stream)))
        return o

    def group_forward(self, slot: int, hidden: torch.Tensor, tokens: torch.Tensor, top_n: int = 1,
                      want_logits: bool = True, want_feat: bool = False, stream=None) -> dict:
        """ps_group_forward: the group-wise training layout, forward only.  hidden [n][H], tokens
        [n] int32; outputs shaped [n][k+1]..."""
        n, R, V, H = tokens.shape[0], self.rows, self.cfg.vocab, self.cfg.hidden
        dev = "cuda"
        o = {"top_ids": torch.empty((n, R, max(top_n, 1)), dtype=torch.int32, device=dev),
             "top_logit": torch.empty((n, R, max(top_n, 1)), dtype=torch.float32, device=dev),
             "row_max": torch.empty((n, R), dtype=torch.float32, device=dev),
             "row_lse": torch.empty((n, R), dtype=torch.float32, device=dev),
             "logits": torch.empty((n, R, V), dtype=torch.float32, device=dev) if want_logits else None,
             "feat": torch.empty((n, R, H), dtype=torch.float32, device=dev) if want_feat else None}
        self._check(self.lib.ps_group_forward(
            self.h, slot, n, _dptr(hidden), _dptr(tokens), top_n, _dptr(o["top_ids"]), _dptr(o["top_logit"]),
            _dptr(o["row_max"]), _dptr(o["row_lse"]), _dptr(o["logits"]), _dptr(o["feat"]), _stream(stream)))
        return o

    def draft_step_sampled(self, seq_slot, hidden_last: torch.Tensor, token_last: torch.Tensor,
                           temperature: float, seed: int, offset: int, top_n: int = 1,
                           want_logits: bool = True, want_feat: bool = False, out: dict | None = None,
                           stream=None) -> dict:
        """ps_draft_step_sampled: ps_draft_step plus ``sampled`` [B][k+1] int32, one token per row
        drawn from softmax(logits / temperature)."""
        B, R, V, H = len(seq_slot), self.rows, self.cfg.vocab, self.cfg.hidden
        o = out if out is not None else {}
        dev = "cuda"
        if "row_max" not in o:
            o["top_ids"] = torch.empty((B, R, max(top_n, 1)), dtype=torch.int32, device=dev)
            o["top_logit"] = torch.empty((B, R, max(top_n, 1)), dtype=torch.float32, device=dev)
            o["row_max"] = torch.empty((B, R), dtype=torch.float32, device=dev)
            o["row_lse"] = torch.empty((B, R), dtype=torch.float32, device=dev)
            o["logits"] = torch.empty((B, R, V), dtype=torch.float32, device=dev) if want_logits else None
            o["feat"] = torch.empty((B, R, H), dtype=torch.float32, device=dev) if want_feat else None
        if "sampled" not in o:
            o["sampled"] = torch.empty((B, R), dtype=torch.int32, device=dev)
        self._check(self.lib.ps_draft_step_sampled(
            self.h, B, _iarr(seq_slot), _dptr(hidden_last), _dptr(token_last), float(temperature), seed, offset,
            _dptr(o["sampled"]), top_n, _dptr(o["top_ids"]), _dptr(o["top_logit"]), _dptr(o["row_max"]),
            _dptr(o["row_lse"]), _dptr(o.get("logits")), _dptr(o.get("feat")), _stream(stream)))
        return o

    def verify(self, draft_tokens: torch.Tensor, draft_logits, target_logits: torch.Tensor,
               temperature: float, seed: int, offset: int, out: dict | None = None, stream=None) -> dict:
        """ps_verify.  draft_tokens [B][n_draft] int32, target_logits [B][n_target][V] float32."""
        B, n_draft = draft_tokens.shape
        n_target = target_logits.shape[1]
        assert target_logits.shape[2] == self.cfg.vocab and target_logits.dtype == torch.float32
        o = out if out is not None else {}
        if "accept_len" not in o:
            o["accept_len"] = torch.empty(B, dtype=torch.int32, device="cuda")
            o["out_tokens"] = torch.empty((B, n_draft + 1), dtype=torch.int32, device="cuda")
            o["n_out"] = torch.empty(B, dtype=torch.int32, device="cuda")
        self._check(self.lib.ps_verify(
            self.h, B, n_draft, n_target, _dptr(draft_tokens), _dptr(draft_logits),
            _dptr(target_logits), float(temperature), seed, offset, _dptr(o["accept_len"]),
            _dptr(o["out_tokens"]), _dptr(o["n_out"]), _stream(stream)))
        return o

    def verify_tree(self, parent, tokens: torch.Tensor, draft_logits, target_logits: torch.Tensor,
                    temperature: float, seed: int, offset: int, out: dict | None = None, stream=None) -> dict:
        """ps_verify_tree.  parent: host list [n_nodes]; tokens [B][n_nodes] int32; draft_logits
        [B][D][V] float32 (D = 1 + largest depth) or None at temperature 0; target_logits
        [B][n_nodes+1][V] float32."""
        B, n_nodes = tokens.shape
        assert len(parent) == n_nodes and target_logits.shape == (B, n_nodes + 1, self.cfg.vocab)
        depth = []
        for i, p in enumerate(parent):
            depth.append(0 if p < 0 or p >= i else depth[p] + 1)   # a malformed tree is the library's to reject
        D = max(depth) + 1
        if draft_logits is not None:
            assert draft_logits.shape == (B, D, self.cfg.vocab) and draft_logits.dtype == torch.float32
        o = out if out is not None else {}
        if "accept_len" not in o:
            o["accept_len"] = torch.empty(B, dtype=torch.int32, device="cuda")
            o["out_tokens"] = torch.empty((B, D + 1), dtype=torch.int32, device="cuda")
            o["n_out"] = torch.empty(B, dtype=torch.int32, device="cuda")
            o["path"] = torch.empty((B, D), dtype=torch.int32, device="cuda")
        self._check(self.lib.ps_verify_tree(
            self.h, B, n_nodes, _iarr(parent), _dptr(tokens), _dptr(draft_logits), _dptr(target_logits),
            float(temperature), seed, offset, _dptr(o["accept_len"]), _dptr(o["out_tokens"]),
            _dptr(o["n_out"]), _dptr(o["path"]), _stream(stream)))
        return o

    def build_tree(self, parent, rank, top_ids: torch.Tensor, sampled_ids=None, out=None, stream=None):
        """ps_build_tree.  parent, rank: host lists [n_nodes]; top_ids [B][k+1][top_n] int32 (a draft
        step's output); sampled_ids [B][k+1] int32 or None.  Returns tokens [B][n_nodes] int32."""
        B, R, top_n = top_ids.shape
        assert R == self.rows and top_ids.dtype == torch.int32 and top_ids.is_contiguous()
        n_nodes = len(parent)
        assert len(rank) == n_nodes
        tokens = out if out is not None else torch.empty((B, n_nodes), dtype=torch.int32, device="cuda")
        self._check(self.lib.ps_build_tree(self.h, B, n_nodes, _iarr(parent), _iarr(rank), _dptr(top_ids), top_n,
                                           _dptr(sampled_ids), _dptr(tokens), _stream(stream)))
        return tokens

    def round_host(self, seq_slot, hidden_last: torch.Tensor, token_last: torch.Tensor,
                   target_logits: torch.Tensor, temperature: float, seed: int, offset: int,
                   out: dict | None = None, stream=None) -> dict:
        """ps_round_host: all tensors are HOST tensors (pinned for asynchronous copies)."""
        B, R = len(seq_slot), self.rows
        for t in (hidden_last, token_last, target_logits):
            assert not t.is_cuda and t.is_contiguous()
        o = out if out is not None else {}
        if "accept_len" not in o:
            o["accept_len"] = torch.empty(B, dtype=torch.int32).pin_memory()
            o["out_tokens"] = torch.empty((B, R + 1), dtype=torch.int32).pin_memory()
            o["n_out"] = torch.empty(B, dtype=torch.int32).pin_memory()
        hp = lambda t: C.c_void_p(t.data_ptr())
        self._check(self.lib.ps_round_host(
            self.h, B, _iarr(seq_slot), hp(hidden_last), hp(token_last), hp(target_logits),
            float(temperature), seed, offset, hp(o["accept_len"]), hp(o["out_tokens"]),
            hp(o["n_out"]), _stream(stream)))
        return o

    def check_guards(self, stream=None) -> int:
        """ps_debug_check_guards: number of workspace slices whose guard words were overwritten."""
        n = C.c_int(-1)
        self._check(self.lib.ps_debug_check_guards(self.h, _stream(stream), C.byref(n)))
        return n.value

    def debug_wait_expires(self, limit_cycles: int, stream=None) -> None:
        """ps_debug_wait_expires: a bounded device wait that runs out (sets the status word)."""
        self._check(self.lib.ps_debug_wait_expires(self.h, int(limit_cycles), _stream(stream)))

    def poll(self) -> int:
        """Waits for the stream and returns the device status (PS_OK, PS_ERR_NONFINITE, ...)."""
        return self.lib.ps_poll(self.h, _stream())

    def profile(self, enable) -> None:
        """ps_profile: False / 0 off, True / 1 an event per stage, 2 an event per launch."""
        self._check(self.lib.ps_profile(self.h, int(enable)))

    def profile_read(self) -> dict:
        """{stage: (total_ms, intervals)} since profiling was enabled or last read."""
        n_max = 32
        names = C.create_string_buffer(32 * n_max)
        ms = (C.c_float * n_max)()
        cnt = (C.c_int * n_max)()
        n = C.c_int()
        self._check(self.lib.ps_profile_read(self.h, n_max, names, ms, cnt, C.byref(n)))
        raw = names.raw
        return {raw[32 * i:32 * i + 32].split(b"\0")[0].decode(): (ms[i], cnt[i]) for i in range(n.value)}

    def debug_buffer(self, name: str, dtype, shape) -> torch.Tensor:
        """Copy of an intermediate buffer of the last draft step (test helper)."""
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        self._check(self.lib.ps_debug_buffer(self.h, name.encode(), C.byref(ptr), C.byref(nbytes)))
        base = self.workspace.data_ptr()
        off = ptr.value - base
        n = 1
        for d in shape:
            n *= d
        elt = torch.empty((), dtype=dtype).element_size()
        assert 0 <= off and n * elt <= nbytes.value and off + n * elt <= self.workspace.numel()
        return self.workspace[off:off + n * elt].view(dtype).view(*shape).clone()

    def launch_count(self) -> int:
        return self.lib.ps_launch_count(self.h)
