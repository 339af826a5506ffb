"""Thin ctypes binding of the trimkv C ABI (include/trimkv.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  torch tensors
supply device memory and the current stream.  There is no CPU fallback: if the shared library has not
been built, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtrimkv.so")

OK, E_ARG, E_STATE, E_NOMEM, E_CUDA, E_NONFINITE, E_TIMEOUT, E_UNSUPPORTED = range(8)
STATUS_NAMES = ["OK", "E_ARG", "E_STATE", "E_NOMEM", "E_CUDA", "E_NONFINITE", "E_TIMEOUT", "E_UNSUPPORTED"]
DTYPE_BF16, DTYPE_F32 = 0, 1
TEST_DISTRUST_SAMPLE, TEST_ATTENTION_NO_COPY = 1, 2     # testing aids, see trimkv_set_test_hooks

EXPORTS = [
    "trimkv_default_config", "trimkv_create", "trimkv_create_ex", "trimkv_destroy", "trimkv_reset", "trimkv_set_gate",
    "trimkv_set_shared_projection", "trimkv_gate", "trimkv_append", "trimkv_score_and_evict", "trimkv_decode_attention",
    "trimkv_prefill_attention", "trimkv_decode_step_all", "trimkv_decode_step_all_host", "trimkv_get_lengths", "trimkv_get_kept", "trimkv_get_pool", "trimkv_get_select_stats",
    "trimkv_sync_status", "trimkv_set_overlap", "trimkv_set_horizon", "trimkv_profile", "trimkv_profile_read", "trimkv_last_error", "trimkv_kernel_launches", "trimkv_select_workspace_bytes",
    "trimkv_select_topk", "trimkv_select_topk_static", "trimkv_set_test_hooks",
    "trimkv_step_stream", "trimkv_check_invariants", "trimkv_import_pool", "trimkv_import_finish", "trimkv_shard_sample_cap", "trimkv_shard_sample", "trimkv_shard_bracket", "trimkv_shard_filter", "trimkv_shard_candidates",
    "trimkv_shard_resolve", "trimkv_shard_hist", "trimkv_shard_digit", "trimkv_shard_mark", "trimkv_shard_compact",
]


class TrimkvError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"trimkv {STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}: {message}")
        self.status = status


class Config(C.Structure):
    _fields_ = [
        ("budget_entries", C.c_int64), ("layers", C.c_int32), ("kv_heads", C.c_int32), ("q_heads", C.c_int32),
        ("head_dim", C.c_int32), ("hidden", C.c_int32), ("max_batch", C.c_int32), ("page_size", C.c_int32),
        ("gate_hidden", C.c_int32), ("gate_embed", C.c_int32), ("horizon", C.c_int32), ("kv_dtype", C.c_int32),
        ("max_chunk", C.c_int32), ("reserved", C.c_int32), ("max_pool_pages", C.c_int64),
        ("retention_bias", C.c_int32), ("per_pool_budget", C.c_int32),
        ("shard_total_layers", C.c_int32), ("shard_layer0", C.c_int32),
    ]


_lib = None


def lib() -> C.CDLL:
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_09649_b200.build` "
                           "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_float
    L.trimkv_default_config.argtypes = [C.POINTER(Config), i64, i32, i32, i32]
    L.trimkv_default_config.restype = None
    L.trimkv_create.argtypes = [i64, i32, i32, i32]
    L.trimkv_create.restype = vp
    L.trimkv_create_ex.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    L.trimkv_destroy.argtypes = [vp]
    L.trimkv_destroy.restype = None
    L.trimkv_reset.argtypes = [vp]
    L.trimkv_set_gate.argtypes = [vp, i32, vp, vp, vp, vp]
    L.trimkv_set_shared_projection.argtypes = [vp, vp, f32]
    L.trimkv_gate.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    L.trimkv_append.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
    L.trimkv_score_and_evict.argtypes = [vp, vp]
    L.trimkv_decode_attention.argtypes = [vp, i32, vp, vp, vp]
    L.trimkv_prefill_attention.argtypes = [vp, i32, i32, vp, vp, vp]
    L.trimkv_prefill_attention.restype = i32
    L.trimkv_decode_step_all.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    L.trimkv_decode_step_all_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    L.trimkv_decode_step_all_host.restype = i32
    L.trimkv_get_lengths.argtypes = [vp, vp]
    L.trimkv_get_kept.argtypes = [vp, i32, i32, i32, vp, i32, C.POINTER(i32)]
    L.trimkv_get_pool.argtypes = [vp, i32, i32, i32, i32, C.POINTER(i32), vp, vp, vp, vp, vp]
    L.trimkv_get_select_stats.argtypes = [vp, vp]
    L.trimkv_sync_status.argtypes = [vp]
    L.trimkv_profile.argtypes = [vp, i32]
    L.trimkv_set_overlap.argtypes = [vp, i32]
    L.trimkv_set_test_hooks.argtypes = [vp, i32]
    L.trimkv_step_stream.argtypes = [vp]
    L.trimkv_check_invariants.argtypes = [vp]
    L.trimkv_check_invariants.restype = i32
    L.trimkv_import_pool.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp]
    L.trimkv_import_pool.restype = i32
    L.trimkv_import_finish.argtypes = [vp, i64]
    L.trimkv_import_finish.restype = i32
    L.trimkv_step_stream.restype = vp
    L.trimkv_shard_sample_cap.argtypes = []
    L.trimkv_shard_sample.argtypes = [vp, i64, i64, vp, vp, vp]
    L.trimkv_shard_bracket.argtypes = [vp, i32, vp, vp, i64, i64, vp]
    L.trimkv_shard_filter.argtypes = [vp, vp, vp, vp]
    L.trimkv_shard_candidates.argtypes = [vp, i64, vp, vp]
    L.trimkv_shard_resolve.argtypes = [vp, i32, i32, i64, vp, vp, vp, i64, vp, vp]
    L.trimkv_shard_hist.argtypes = [vp, vp, i32, vp, vp]
    L.trimkv_shard_digit.argtypes = [vp, vp, vp, vp, i32, vp]
    L.trimkv_shard_mark.argtypes = [vp, vp, vp]
    L.trimkv_shard_compact.argtypes = [vp, vp, vp]
    L.trimkv_set_horizon.argtypes = [vp, i32, vp]
    L.trimkv_profile_read.argtypes = [vp, vp, vp]
    L.trimkv_last_error.argtypes = []
    L.trimkv_last_error.restype = C.c_char_p
    L.trimkv_kernel_launches.argtypes = []
    L.trimkv_kernel_launches.restype = i64
    L.trimkv_select_workspace_bytes.argtypes = [i64]
    L.trimkv_select_workspace_bytes.restype = C.c_size_t
    L.trimkv_select_topk.argtypes = [vp, i64, i64, vp, vp, C.c_size_t, vp, vp]
    L.trimkv_select_topk_static.argtypes = [vp, i64, i64, vp, vp, vp]
    for name in ("trimkv_create_ex", "trimkv_reset", "trimkv_set_gate", "trimkv_set_shared_projection", "trimkv_gate",
                 "trimkv_append", "trimkv_score_and_evict", "trimkv_decode_attention", "trimkv_decode_step_all",
                 "trimkv_get_lengths", "trimkv_get_kept", "trimkv_get_pool", "trimkv_get_select_stats",
                 "trimkv_sync_status", "trimkv_profile", "trimkv_profile_read", "trimkv_select_topk",
                 "trimkv_select_topk_static", "trimkv_set_overlap", "trimkv_set_horizon", "trimkv_set_test_hooks",
                 "trimkv_shard_sample_cap", "trimkv_shard_sample", "trimkv_shard_bracket", "trimkv_shard_filter",
                 "trimkv_shard_candidates", "trimkv_shard_resolve", "trimkv_shard_hist", "trimkv_shard_digit",
                 "trimkv_shard_mark", "trimkv_shard_compact"):
        getattr(L, name).restype = i32
    _lib = L
    return L


def last_error() -> str:
    return lib().trimkv_last_error().decode("utf-8", "replace")


def kernel_launches() -> int:
    return int(lib().trimkv_kernel_launches())


def _check(status: int):
    if status != OK:
        raise TrimkvError(status, last_error())


def _ptr(t: Optional[torch.Tensor], dtype=None, cuda=True):
    if t is None:
        return None
    if cuda and not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class TrimKV:
    """One budgeted, paged KV cache for a fixed batch of sequences (see include/trimkv.h)."""

    def __init__(self, budget_entries: int, layers: int, kv_heads: int, head_dim: int, *, q_heads: Optional[int] = None,
                 hidden: int = 0, batch: int = 1, gate_hidden: int = 512, gate_embed: int = 64, horizon: int = 2,
                 kv_dtype: str = "bf16", max_chunk: int = 512, max_pool_pages: int = 0, distrust_sample: bool = False,
                 retention_bias: bool = False, per_pool_budget: int = 0, shard_total_layers: int = 0, shard_layer0: int = 0):
        L = lib()
        cfg = Config()
        L.trimkv_default_config(C.byref(cfg), budget_entries, layers, kv_heads, head_dim)
        cfg.q_heads = q_heads if q_heads is not None else kv_heads
        cfg.hidden = hidden
        cfg.max_batch = batch
        cfg.gate_hidden = gate_hidden
        cfg.gate_embed = gate_embed
        cfg.horizon = horizon
        cfg.kv_dtype = {"bf16": DTYPE_BF16, "f32": DTYPE_F32}[kv_dtype]
        cfg.max_chunk = max_chunk
        cfg.max_pool_pages = max_pool_pages
        cfg.retention_bias = 1 if retention_bias else 0
        cfg.per_pool_budget = per_pool_budget
        cfg.shard_total_layers = shard_total_layers
        cfg.shard_layer0 = shard_layer0
        cfg.reserved = 0
        self.cfg = cfg
        self.torch_dtype = torch.bfloat16 if kv_dtype == "bf16" else torch.float32
        self.B, self.L, self.H, self.Hq, self.d, self.D = batch, layers, kv_heads, cfg.q_heads, head_dim, hidden
        h = C.c_void_p()
        _check(L.trimkv_create_ex(C.byref(cfg), C.byref(h)))
        self._h = h
        if distrust_sample:                            # testing aid: forces the selection's exact redo path
            self.set_test_hooks(TEST_DISTRUST_SAMPLE)

    @classmethod
    def from_workload(cls, w, **overrides) -> "TrimKV":
        kw = dict(q_heads=w.q_heads, hidden=w.hidden, batch=w.batch, gate_hidden=w.gate_hidden, gate_embed=w.gate_embed,
                  horizon=w.horizon, kv_dtype=w.kv_dtype, max_chunk=w.chunk)
        kw.update(overrides)
        return cls(w.budget_entries, w.layers, w.kv_heads, w.head_dim, **kw)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib().trimkv_destroy(self._h)
            self._h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    # ---- gate
    def set_gate(self, layer: int, W1, b1, W2, b2):
        f = torch.float32
        _check(lib().trimkv_set_gate(self._h, layer, _ptr(W1, f), _ptr(b1, f), _ptr(W2, f), _ptr(b2, f)))

    def set_shared_projection(self, w_g, b_g: float):
        _check(lib().trimkv_set_shared_projection(self._h, _ptr(w_g, torch.float32), float(b_g)))

    def gate(self, layer: int, x: torch.Tensor):
        """x [B, n, D] fp32 -> (beta, lambda, c), each [B, n, H] fp32."""
        n = x.shape[1]
        outs = [torch.empty(self.B, n, self.H, device=x.device, dtype=torch.float32) for _ in range(3)]
        _check(lib().trimkv_gate(self._h, layer, n, _ptr(x, torch.float32), _ptr(outs[0]), _ptr(outs[1]), _ptr(outs[2]),
                                 _stream()))
        return tuple(outs)

    # ---- cache
    def append(self, layer: int, k, v, x=None, lam=None, c=None):
        n = k.shape[1]
        f = torch.float32
        _check(lib().trimkv_append(self._h, layer, n, _ptr(x, f), _ptr(lam, f), _ptr(c, f), _ptr(k, self.torch_dtype),
                                   _ptr(v, self.torch_dtype), _stream()))

    def score_and_evict(self):
        _check(lib().trimkv_score_and_evict(self._h, _stream()))

    def decode_attention(self, layer: int, q, out=None):
        if out is None:
            out = torch.empty_like(q)
        _check(lib().trimkv_decode_attention(self._h, layer, _ptr(q, self.torch_dtype), _ptr(out, self.torch_dtype),
                                             _stream()))
        return out

    def prefill_attention(self, layer: int, q, out=None):
        """q [B, n, Hq, d]: causal attention of the n-token chunk just appended to `layer`."""
        if out is None:
            out = torch.empty_like(q)
        _check(lib().trimkv_prefill_attention(self._h, layer, q.shape[1], _ptr(q, self.torch_dtype),
                                              _ptr(out, self.torch_dtype), _stream()))
        return out

    def decode_step_all(self, k, v, q, out, x=None, lam=None):
        f = torch.float32
        _check(lib().trimkv_decode_step_all(self._h, _ptr(x, f), _ptr(lam, f), _ptr(k, self.torch_dtype),
                                            _ptr(v, self.torch_dtype), _ptr(q, self.torch_dtype),
                                            _ptr(out, self.torch_dtype), _stream()))
        return out

    def decode_step_all_host(self, k, v, q, out, x=None, lam=None):
        """Same step with HOST tensors (pinned for asynchronous copies); `out` is a host tensor as well."""
        f = torch.float32
        _check(lib().trimkv_decode_step_all_host(self._h, _ptr(x, f, cuda=False), _ptr(lam, f, cuda=False),
                                                 _ptr(k, self.torch_dtype, cuda=False), _ptr(v, self.torch_dtype, cuda=False),
                                                 _ptr(q, self.torch_dtype, cuda=False), _ptr(out, self.torch_dtype, cuda=False),
                                                 _stream()))
        return out

    def reset(self):
        _check(lib().trimkv_reset(self._h))

    def sync_status(self):
        _check(lib().trimkv_sync_status(self._h))

    def check_invariants(self):
        """Self-check of the cache's bookkeeping (raises TrimkvError E_STATE naming the violated rules)."""
        _check(lib().trimkv_check_invariants(self._h))

    PHASES = ["gate", "append", "h2d_kvq", "attn_main", "d2h_out", "select", "compact", "h2d_x"]

    def profile(self, enable):
        """False/0 off, True/1 every phase, 2 the attention kernel alone."""
        _check(lib().trimkv_profile(self._h, int(enable)))

    def set_horizon(self, horizon: int):
        """New horizon T - t for stored and future entries (0 = infinite)."""
        _check(lib().trimkv_set_horizon(self._h, int(horizon), _stream()))

    def set_test_hooks(self, flags: int):
        """Testing aids of this handle (TEST_* flags; 0 = normal operation)."""
        _check(lib().trimkv_set_test_hooks(self._h, int(flags)))

    def step_stream(self) -> "torch.cuda.ExternalStream":
        """The handle's highest-priority stream as a torch stream: decode steps enqueued on it skip two stream hand-offs."""
        return torch.cuda.ExternalStream(int(lib().trimkv_step_stream(self._h)))

    def set_overlap(self, enable: bool):
        _check(lib().trimkv_set_overlap(self._h, 1 if enable else 0))

    def profile_read(self):
        """{phase: (total ms, intervals)} recorded since profiling was enabled."""
        ms = (C.c_double * 8)()
        cnt = (C.c_int64 * 8)()
        _check(lib().trimkv_profile_read(self._h, ms, cnt))
        return {name: (ms[i], cnt[i]) for i, name in enumerate(self.PHASES)}

    # ---- read-back (synchronising)
    def lengths(self) -> torch.Tensor:
        out = torch.empty(self.B, self.L, self.H, dtype=torch.int32)
        _check(lib().trimkv_get_lengths(self._h, C.c_void_p(out.data_ptr())))
        return out

    def kept(self, seq: int, layer: int, head: int, cap: int) -> torch.Tensor:
        out = torch.empty(max(cap, 1), dtype=torch.int32)
        n = C.c_int(0)
        _check(lib().trimkv_get_kept(self._h, seq, layer, head, C.c_void_p(out.data_ptr()), cap, C.byref(n)))
        return out[: n.value].clone()

    def pool(self, seq: int, layer: int, head: int, cap: int, with_kv: bool = True):
        pos = torch.empty(max(cap, 1), dtype=torch.int32)
        lam = torch.empty(max(cap, 1), dtype=torch.float32)
        c = torch.empty(max(cap, 1), dtype=torch.float32)
        k = torch.empty(max(cap, 1), self.d, dtype=self.torch_dtype) if with_kv else None
        v = torch.empty(max(cap, 1), self.d, dtype=self.torch_dtype) if with_kv else None
        n = C.c_int(0)
        _check(lib().trimkv_get_pool(self._h, seq, layer, head, cap, C.byref(n), C.c_void_p(pos.data_ptr()),
                                     C.c_void_p(lam.data_ptr()), C.c_void_p(c.data_ptr()),
                                     C.c_void_p(k.data_ptr()) if with_kv else None,
                                     C.c_void_p(v.data_ptr()) if with_kv else None))
        m = n.value
        return pos[:m], lam[:m], c[:m], (k[:m] if with_kv else None), (v[:m] if with_kv else None)

    def import_pool(self, seq: int, layer: int, head: int, pos, lam, c, k, v):
        """Fills the (empty) pool from host tensors as `pool` returned them (checkpoint resume)."""
        n = int(pos.numel())
        hp = lambda t: C.c_void_p(t.contiguous().data_ptr()) if n else None
        _check(lib().trimkv_import_pool(self._h, seq, layer, head, n, hp(pos), hp(lam), hp(c), hp(k), hp(v)))

    def import_finish(self, tokens: int):
        _check(lib().trimkv_import_finish(self._h, int(tokens)))

    def select_stats(self) -> torch.Tensor:
        out = torch.empty(self.B, 4, dtype=torch.int64)
        _check(lib().trimkv_get_select_stats(self._h, C.c_void_p(out.data_ptr())))
        return out


def set_global_test_hooks(flags: int):
    """Testing aids of the handle-less calls (select_topk, select_topk_static); 0 = normal operation."""
    _check(lib().trimkv_set_test_hooks(None, int(flags)))


def select_workspace_bytes(n: int) -> int:
    return int(lib().trimkv_select_workspace_bytes(n))


def select_topk(scores: torch.Tensor, k_keep: int, keep_bits: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None):
    """Keep mask (uint64 words as int64 tensor) of the k_keep largest fp32 scores; ties keep the lower index."""
    n = scores.numel()
    words = (n + 63) // 64
    if keep_bits is None:
        keep_bits = torch.empty(max(words, 1), dtype=torch.int64, device=scores.device)
    need = select_workspace_bytes(n)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=scores.device)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=scores.device)
    _check(lib().trimkv_select_topk(_ptr(scores, torch.float32), n, k_keep, _ptr(keep_bits), _ptr(workspace),
                                    workspace.numel(), _ptr(status), _stream()))
    return keep_bits, status


SELECT_STATIC_MAX_N = 1 << 22


def select_topk_static(scores: torch.Tensor, k_keep: int, keep_bits: torch.Tensor, status: torch.Tensor):
    """trimkv_select_topk_static: the same selection, for callers that cannot allocate device memory when
    they call (a serving loop with a fixed memory plan, a framework that bans cudaMalloc after start-up).
    The scratch lives inside the library; the caller passes every buffer: keep_bits (int64 words,
    ceil(n / 64) of them) and status (int32[1]).  At most SELECT_STATIC_MAX_N scores.  Calls share the
    scratch, so do not let two of them overlap on the GPU."""
    n = scores.numel()
    _check(lib().trimkv_select_topk_static(_ptr(scores, torch.float32), n, k_keep, _ptr(keep_bits), _ptr(status),
                                           _stream()))
    return keep_bits, status
