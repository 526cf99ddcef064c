"""Thin binding over the C-ABI CUDA library (``libqp.so``): argument marshalling only.

Every function has the name and the meaning of the C entry point it forwards to
(see ``include/qp.h``).  torch is used for device memory, pointers and the current
stream; no step of the path runs in Python or on the CPU.  Loading fails loudly
when the library has not been built.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# QP_LIBRARY selects another build of the same library (the range-checked debug build libqp_checked.so)
LIB_PATH = os.environ.get("QP_LIBRARY") or os.path.join(_HERE, "libqp.so")

QP_OK = 0
QP_MAX_LAYERS = 128
STATUS_NAMES = {0: "QP_OK", 1: "QP_ERR_INVALID_ARG", 2: "QP_ERR_UNSUPPORTED", 3: "QP_ERR_BUDGET",
                4: "QP_ERR_WORKSPACE", 5: "QP_ERR_ALIGNMENT", 6: "QP_ERR_CUDA"}

EXPORTS = ["qp_status_string", "qp_n_keep", "qp_cache_layout", "qp_compress_workspace_bytes",
           "qp_decode_workspace_bytes", "qp_window_scores", "qp_select_topk", "qp_gather_quantize",
           "qp_compress_layer", "qp_decode_attn", "qp_decode_attn_layers", "qp_decode_attn_static",
           "qp_cache_layout_cap", "qp_append_kv", "qp_append_kv_layers", "qp_decode_attn_tail",
           "qp_decode_attn_tail_layers", "qp_compress_layers", "qp_decode_overlap", "qp_gather_quantize_ex",
           "qp_decode_attn_ex", "qp_decode_attn_layers_ex", "qp_head_budgets", "qp_head_budgets_workspace_bytes", "qp_debug_check"]


class QpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({status_string(status)})")


class qp_cache(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("bits", ctypes.c_int32), ("group", ctypes.c_int32),
                ("n_keep", ctypes.c_int32), ("n_cap", ctypes.c_int32),
                ("k_codes_bytes", ctypes.c_size_t), ("v_codes_bytes", ctypes.c_size_t),
                ("k_meta_bytes", ctypes.c_size_t), ("v_meta_bytes", ctypes.c_size_t),
                ("k_codes", ctypes.c_void_p), ("v_codes", ctypes.c_void_p),
                ("k_scale", ctypes.c_void_p), ("k_zero", ctypes.c_void_p),
                ("v_scale", ctypes.c_void_p), ("v_zero", ctypes.c_void_p)]


class qp_side(ctypes.Structure):
    _fields_ = [("cap", ctypes.c_int32), ("reserved_", ctypes.c_int32), ("idx", ctypes.c_void_p),
                ("val", ctypes.c_void_p), ("cnt", ctypes.c_void_p), ("tile_ptr", ctypes.c_void_p)]


class qp_strategy(ctypes.Structure):
    _fields_ = [("k_axis", ctypes.c_int32), ("outlier_threshold", ctypes.c_float),
                ("k_side", qp_side), ("v_side", qp_side)]


class qp_tail(ctypes.Structure):
    _fields_ = [("n_tail", ctypes.c_int32), ("reserved_", ctypes.c_int32),
                ("k_tail", ctypes.c_void_p), ("v_tail", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded CUDA library.  Raises if it is missing: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2412_12706_b200.build` (needs nvcc, sm_100a)")
        L = ctypes.CDLL(LIB_PATH)
        i, i64, p, sz = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t
        cp = ctypes.POINTER(qp_cache)
        L.qp_status_string.restype = ctypes.c_char_p
        L.qp_status_string.argtypes = [i]
        L.qp_n_keep.restype = i
        L.qp_n_keep.argtypes = [i64, i, i, i, i, ctypes.POINTER(ctypes.c_int32)]
        L.qp_cache_layout.restype = i
        L.qp_cache_layout.argtypes = [i, i, i, i, i, i, i, cp]
        L.qp_compress_workspace_bytes.restype = sz
        L.qp_compress_workspace_bytes.argtypes = [i, i, i, i, i, i]
        L.qp_decode_workspace_bytes.restype = sz
        L.qp_decode_workspace_bytes.argtypes = [cp]
        L.qp_window_scores.restype = i
        L.qp_window_scores.argtypes = [p, p, i, i, i, i, i, i, i, p, p, sz, p]
        L.qp_select_topk.restype = i
        L.qp_select_topk.argtypes = [p, i, i, i, i, i, p, p]
        L.qp_gather_quantize.restype = i
        L.qp_gather_quantize.argtypes = [p, p, p, i, cp, p]
        L.qp_compress_layer.restype = i
        L.qp_compress_layer.argtypes = [p, p, p, i, i, i, i, i, i, i64, i, i, i, cp, p, p, sz, p]
        L.qp_decode_attn.restype = i
        L.qp_decode_attn.argtypes = [p, cp, p, p, sz, p]
        L.qp_decode_attn_layers.restype = i
        L.qp_decode_attn_layers.argtypes = [i, ctypes.POINTER(p), cp, ctypes.POINTER(p), p, sz, p]
        L.qp_decode_attn_static.restype = i
        L.qp_decode_attn_static.argtypes = [p, cp, p, p]
        tp = ctypes.POINTER(qp_tail)
        L.qp_compress_layers.restype = i
        L.qp_compress_layers.argtypes = [i, ctypes.POINTER(p), ctypes.POINTER(p), ctypes.POINTER(p), i, i, i, i, i, i,
                                         ctypes.POINTER(i64), i, i, i, cp, ctypes.POINTER(p), p, sz, p]
        L.qp_cache_layout_cap.restype = i
        L.qp_cache_layout_cap.argtypes = [i, i, i, i, i, i, i, i, cp]
        L.qp_append_kv.restype = i
        L.qp_append_kv.argtypes = [p, p, cp, tp, p]
        L.qp_append_kv_layers.restype = i
        L.qp_append_kv_layers.argtypes = [i, ctypes.POINTER(p), ctypes.POINTER(p), cp, tp, p]
        L.qp_decode_attn_tail.restype = i
        L.qp_decode_attn_tail.argtypes = [p, cp, tp, p, p, sz, p]
        L.qp_decode_attn_tail_layers.restype = i
        L.qp_decode_attn_tail_layers.argtypes = [i, ctypes.POINTER(p), cp, tp, ctypes.POINTER(p), p, sz, p]
        sp = ctypes.POINTER(qp_strategy)
        L.qp_gather_quantize_ex.restype = i
        L.qp_gather_quantize_ex.argtypes = [p, p, p, i, cp, sp, p]
        L.qp_decode_attn_ex.restype = i
        L.qp_decode_attn_ex.argtypes = [p, cp, sp, p, p, sz, p]
        L.qp_decode_attn_layers_ex.restype = i
        L.qp_decode_attn_layers_ex.argtypes = [i, ctypes.POINTER(p), cp, sp, ctypes.POINTER(p), p, sz, p]
        L.qp_head_budgets_workspace_bytes.restype = sz
        L.qp_head_budgets_workspace_bytes.argtypes = [i, i, i, i, i]
        L.qp_head_budgets.restype = i
        L.qp_head_budgets.argtypes = [p, i, i, i, i, i, i, p, p, sz, p]
        L.qp_debug_check.restype = i
        L.qp_debug_check.argtypes = [ctypes.POINTER(ctypes.c_uint32)]
        L.qp_decode_overlap.restype = i
        L.qp_decode_overlap.argtypes = [p, i]
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != QP_OK:
        raise QpError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: torch.Tensor | None) -> int | None:
    return None if t is None else t.data_ptr()


def status_string(status: int) -> str:
    return lib().qp_status_string(status).decode()


def n_keep(budget_bits: int, bits: int, group: int, L: int, w: int) -> int:
    out = ctypes.c_int32(0)
    _check(lib().qp_n_keep(budget_bits, bits, group, L, w, ctypes.byref(out)), "qp_n_keep")
    return out.value


def cache_layout(batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, bits: int, group: int,
                 n_keep_: int) -> qp_cache:
    c = qp_cache()
    _check(lib().qp_cache_layout(batch, n_q_heads, n_kv_heads, head_dim, bits, group, n_keep_,
                                 ctypes.byref(c)), "qp_cache_layout")
    return c


def cache_layout_cap(batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, bits: int, group: int,
                     n_keep_: int, n_cap: int) -> qp_cache:
    c = qp_cache()
    _check(lib().qp_cache_layout_cap(batch, n_q_heads, n_kv_heads, head_dim, bits, group, n_keep_, n_cap,
                                     ctypes.byref(c)), "qp_cache_layout_cap")
    return c


def compress_workspace_bytes(batch, n_q_heads, n_kv_heads, head_dim, L, w) -> int:
    return int(lib().qp_compress_workspace_bytes(batch, n_q_heads, n_kv_heads, head_dim, L, w))


def decode_workspace_bytes(cache: "Cache | qp_cache") -> int:
    c = cache.desc if isinstance(cache, Cache) else cache
    return int(lib().qp_decode_workspace_bytes(ctypes.byref(c)))


@dataclass
class Cache:
    """Device buffers of one layer's packed cache plus the C descriptor that points at them."""
    desc: qp_cache
    k_codes: torch.Tensor
    v_codes: torch.Tensor
    k_scale: torch.Tensor | None
    k_zero: torch.Tensor | None
    v_scale: torch.Tensor | None
    v_zero: torch.Tensor | None

    @property
    def nbytes(self) -> int:
        d = self.desc
        return d.k_codes_bytes + d.v_codes_bytes + 2 * d.k_meta_bytes + 2 * d.v_meta_bytes


def alloc_cache(batch, n_q_heads, n_kv_heads, head_dim, bits, group, n_keep_, device="cuda",
                n_cap: int = 0) -> Cache:
    """Allocates the buffers of ``qp_cache_layout`` (``qp_cache_layout_cap`` when ``n_cap`` leaves room
    for appended tokens) with torch and fills in the pointers."""
    d = cache_layout_cap(batch, n_q_heads, n_kv_heads, head_dim, bits, group, n_keep_, n_cap)
    n, D, g = (n_cap or n_keep_), head_dim, group
    if bits == 16:
        kc = torch.empty((batch, n_kv_heads, n, D), dtype=torch.bfloat16, device=device)
        vc = torch.empty_like(kc)
        ks = kz = vs = vz = None
    else:
        wpg = g * bits // 32
        kc = torch.empty((batch, n_kv_heads, n // g, D, wpg), dtype=torch.int32, device=device)
        vc = torch.empty((batch, n_kv_heads, n, D // g, wpg), dtype=torch.int32, device=device)
        ks = torch.empty((batch, n_kv_heads, n // g, D), dtype=torch.float16, device=device)
        kz = torch.empty_like(ks)
        vs = torch.empty((batch, n_kv_heads, n, D // g), dtype=torch.float16, device=device)
        vz = torch.empty_like(vs)
    assert kc.numel() * kc.element_size() == d.k_codes_bytes and vc.numel() * vc.element_size() == d.v_codes_bytes
    d.k_codes, d.v_codes = _ptr(kc), _ptr(vc)
    d.k_scale, d.k_zero, d.v_scale, d.v_zero = _ptr(ks), _ptr(kz), _ptr(vs), _ptr(vz)
    return Cache(d, kc, vc, ks, kz, vs, vz)


def _dims(K: torch.Tensor, Q_win: torch.Tensor):
    Bt, Hkv, L, D = K.shape
    _, Hq, w, _ = Q_win.shape
    return Bt, Hq, Hkv, D, L, w


def _dev_bf16(t: torch.Tensor) -> None:
    assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()


def window_scores(Q_win: torch.Tensor, K: torch.Tensor, pool: int = 7, workspace: torch.Tensor | None = None,
                  scores: torch.Tensor | None = None) -> torch.Tensor:
    _dev_bf16(Q_win); _dev_bf16(K)
    Bt, Hq, Hkv, D, L, w = _dims(K, Q_win)
    if scores is None:
        scores = torch.empty((Bt, Hkv, L - w), dtype=torch.float32, device=K.device)
    if workspace is None:
        workspace = torch.empty(max(16, compress_workspace_bytes(Bt, Hq, Hkv, D, L, w)), dtype=torch.uint8,
                                device=K.device)
    _check(lib().qp_window_scores(_ptr(Q_win), _ptr(K), Bt, Hq, Hkv, D, L, w, pool, _ptr(scores),
                                  _ptr(workspace), workspace.numel(), _stream()), "qp_window_scores")
    return scores


def select_topk(scores: torch.Tensor, L: int, w: int, n_keep_: int,
                kept_idx: torch.Tensor | None = None) -> torch.Tensor:
    assert scores.is_cuda and scores.dtype == torch.float32 and scores.is_contiguous()
    Bt, Hkv, P = scores.shape
    assert P == L - w
    if kept_idx is None:
        kept_idx = torch.empty((Bt, Hkv, n_keep_), dtype=torch.int32, device=scores.device)
    _check(lib().qp_select_topk(_ptr(scores), Bt, Hkv, L, w, n_keep_, _ptr(kept_idx), _stream()),
           "qp_select_topk")
    return kept_idx


def gather_quantize(K: torch.Tensor, V: torch.Tensor, kept_idx: torch.Tensor, cache: Cache) -> Cache:
    _dev_bf16(K); _dev_bf16(V)
    assert kept_idx.is_cuda and kept_idx.dtype == torch.int32 and kept_idx.is_contiguous()
    _check(lib().qp_gather_quantize(_ptr(K), _ptr(V), _ptr(kept_idx), K.shape[2], ctypes.byref(cache.desc),
                                    _stream()), "qp_gather_quantize")
    return cache


def compress_layer(K: torch.Tensor, V: torch.Tensor, Q_win: torch.Tensor, budget_bits: int, bits: int,
                   group: int = 32, pool: int = 7, cache: Cache | None = None,
                   kept_idx: torch.Tensor | None = None, workspace: torch.Tensor | None = None, n_cap: int = 0):
    """qp_compress_layer: returns (cache, kept_idx).  Buffers are allocated with torch when not given
    (with room for ``n_cap`` tokens per KV head when ``n_cap`` is given)."""
    _dev_bf16(K); _dev_bf16(V); _dev_bf16(Q_win)
    Bt, Hq, Hkv, D, L, w = _dims(K, Q_win)
    n = n_keep(budget_bits, bits, group, L, w)
    if cache is None:
        cache = alloc_cache(Bt, Hq, Hkv, D, bits, group, n, K.device, n_cap)
    if kept_idx is None:
        kept_idx = torch.empty((Bt, Hkv, n), dtype=torch.int32, device=K.device)
    if workspace is None:
        workspace = torch.empty(max(16, compress_workspace_bytes(Bt, Hq, Hkv, D, L, w)), dtype=torch.uint8,
                                device=K.device)
    _check(lib().qp_compress_layer(_ptr(K), _ptr(V), _ptr(Q_win), Bt, Hq, Hkv, D, L, w, budget_bits, bits,
                                   group, pool, ctypes.byref(cache.desc), _ptr(kept_idx), _ptr(workspace),
                                   workspace.numel(), _stream()), "qp_compress_layer")
    return cache, kept_idx


def compress_layers(Ks: list[torch.Tensor], Vs: list[torch.Tensor], Q_wins: list[torch.Tensor], budget_bits: list[int],
                    bits: int, group: int = 32, pool: int = 7, caches: list[Cache] | None = None,
                    kept_idx: list[torch.Tensor] | None = None, workspace: torch.Tensor | None = None):
    """qp_compress_layers: the prefill-side path of several layers of one shape, one launch per stage.
    Returns (caches, kept_idx); buffers are allocated with torch when not given."""
    nl = len(Ks)
    assert 1 <= nl <= QP_MAX_LAYERS and len(Vs) == nl and len(Q_wins) == nl and len(budget_bits) == nl
    for t in (*Ks, *Vs, *Q_wins):
        _dev_bf16(t)
    Bt, Hq, Hkv, D, L, w = _dims(Ks[0], Q_wins[0])
    ns = [n_keep(b, bits, group, L, w) for b in budget_bits]
    dev = Ks[0].device
    if caches is None:
        caches = [alloc_cache(Bt, Hq, Hkv, D, bits, group, n, dev) for n in ns]
    if kept_idx is None:
        kept_idx = [torch.empty((Bt, Hkv, n), dtype=torch.int32, device=dev) for n in ns]
    if workspace is None:
        workspace = torch.empty(max(16, compress_workspace_bytes(Bt * nl, Hq, Hkv, D, L, w)), dtype=torch.uint8, device=dev)
    arr = lambda ts: (ctypes.c_void_p * nl)(*[t.data_ptr() for t in ts])
    _check(lib().qp_compress_layers(nl, arr(Ks), arr(Vs), arr(Q_wins), Bt, Hq, Hkv, D, L, w,
                                    (ctypes.c_int64 * nl)(*budget_bits), bits, group, pool,
                                    (qp_cache * nl)(*[c.desc for c in caches]), arr(kept_idx), _ptr(workspace),
                                    workspace.numel(), _stream()), "qp_compress_layers")
    return caches, kept_idx


def new_decode_workspace(nbytes: int, device) -> torch.Tensor:
    """Scratch for the decode calls (contents irrelevant); reuse one per stream across calls."""
    return torch.empty(max(16, nbytes), dtype=torch.uint8, device=device)


def decode_attn(q: torch.Tensor, cache: Cache, out: torch.Tensor | None = None,
                workspace: torch.Tensor | None = None) -> torch.Tensor:
    _dev_bf16(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_decode_workspace(decode_workspace_bytes(cache), q.device)
    _check(lib().qp_decode_attn(_ptr(q), ctypes.byref(cache.desc), _ptr(out), _ptr(workspace),
                                workspace.numel(), _stream()), "qp_decode_attn")
    return out


def decode_overlap(enable: bool) -> None:
    """qp_decode_overlap for torch's current stream: let consecutive decode calls on it overlap on the GPU
    (see include/qp.h for what the caller promises while it is on).  Off by default."""
    _check(lib().qp_decode_overlap(_stream(), 1 if enable else 0), "qp_decode_overlap")


class LayerBatch:
    """Marshalled host arrays for ``qp_decode_attn_layers`` (built once, reused every step)."""

    def __init__(self, qs: list[torch.Tensor], caches: list[Cache], outs: list[torch.Tensor],
                 workspace: torch.Tensor | None = None):
        n = len(caches)
        assert 1 <= n <= QP_MAX_LAYERS and len(qs) == n and len(outs) == n
        self.n = n
        self.keep = (qs, caches, outs)
        self.q_arr = (ctypes.c_void_p * n)(*[t.data_ptr() for t in qs])
        self.out_arr = (ctypes.c_void_p * n)(*[t.data_ptr() for t in outs])
        self.cache_arr = (qp_cache * n)(*[c.desc for c in caches])
        if workspace is None:
            workspace = new_decode_workspace(sum(decode_workspace_bytes(c) for c in caches), qs[0].device)
        self.workspace = workspace


def decode_attn_layers(batch: LayerBatch) -> None:
    _check(lib().qp_decode_attn_layers(batch.n, batch.q_arr, batch.cache_arr, batch.out_arr,
                                       _ptr(batch.workspace), batch.workspace.numel(), _stream()),
           "qp_decode_attn_layers")


@dataclass
class Tail:
    """Device buffers of one layer's unquantized tail plus the C descriptor (host state: n_tail)."""
    desc: qp_tail
    k_tail: torch.Tensor | None
    v_tail: torch.Tensor | None


def alloc_tail(cache: Cache, device=None) -> Tail:
    """bf16 [Bt,Hkv,group,D] buffers for the tokens that wait for a full group (none at 16 bit)."""
    d = cache.desc
    t = qp_tail()
    if d.bits == 16:
        return Tail(t, None, None)
    device = device or cache.k_codes.device
    kt = torch.zeros((d.batch, d.n_kv_heads, d.group, d.head_dim), dtype=torch.bfloat16, device=device)
    vt = torch.zeros_like(kt)
    t.k_tail, t.v_tail = _ptr(kt), _ptr(vt)
    return Tail(t, kt, vt)


def append_kv(k_new: torch.Tensor, v_new: torch.Tensor, cache: Cache, tail: Tail) -> None:
    """qp_append_kv: Eq. 2 for one layer; updates cache.desc.n_keep and tail.desc.n_tail."""
    _dev_bf16(k_new); _dev_bf16(v_new)
    _check(lib().qp_append_kv(_ptr(k_new), _ptr(v_new), ctypes.byref(cache.desc), ctypes.byref(tail.desc),
                              _stream()), "qp_append_kv")


def decode_attn_tail(q: torch.Tensor, cache: Cache, tail: Tail, out: torch.Tensor | None = None,
                     workspace: torch.Tensor | None = None) -> torch.Tensor:
    _dev_bf16(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_decode_workspace(decode_workspace_bytes(cache), q.device)
    _check(lib().qp_decode_attn_tail(_ptr(q), ctypes.byref(cache.desc), ctypes.byref(tail.desc), _ptr(out),
                                     _ptr(workspace), workspace.numel(), _stream()), "qp_decode_attn_tail")
    return out


class GenBatch:
    """Marshalled host arrays for a generation loop over many layers: ``qp_append_kv_layers`` followed by
    ``qp_decode_attn_tail_layers``.  The descriptor arrays are owned here and updated in place by the
    append call (the Cache / Tail objects passed in keep their initial descriptors)."""

    def __init__(self, qs, k_news, v_news, caches: list[Cache], tails: list[Tail], outs,
                 workspace: torch.Tensor | None = None):
        n = len(caches)
        assert 1 <= n <= QP_MAX_LAYERS and len(qs) == len(outs) == len(tails) == len(k_news) == len(v_news) == n
        self.n = n
        self.keep = (qs, k_news, v_news, caches, tails, outs)
        arr = lambda ts: (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])
        self.q_arr, self.out_arr, self.kn_arr, self.vn_arr = arr(qs), arr(outs), arr(k_news), arr(v_news)
        self.cache_arr = (qp_cache * n)(*[c.desc for c in caches])
        self.tail_arr = (qp_tail * n)(*[t.desc for t in tails])
        if workspace is None:
            workspace = new_decode_workspace(sum(decode_workspace_bytes(c) for c in caches), qs[0].device)
        self.workspace = workspace


def append_kv_layers(batch: GenBatch) -> None:
    _check(lib().qp_append_kv_layers(batch.n, batch.kn_arr, batch.vn_arr, batch.cache_arr, batch.tail_arr,
                                     _stream()), "qp_append_kv_layers")


def decode_attn_tail_layers(batch: GenBatch) -> None:
    _check(lib().qp_decode_attn_tail_layers(batch.n, batch.q_arr, batch.cache_arr, batch.tail_arr, batch.out_arr,
                                            _ptr(batch.workspace), batch.workspace.numel(), _stream()),
           "qp_decode_attn_tail_layers")


STATIC_SCRATCH_BYTES = 4 << 20


def decode_attn_static(q: torch.Tensor, cache: Cache, out: torch.Tensor | None = None) -> torch.Tensor:
    """qp_decode_attn_static: decode attention whose split partials live in the library's built-in
    scratch array, for hosts that cannot hand the library any temporary device memory.  Only
    ``out`` is allocated here (by torch) when the caller passes none; the C call allocates nothing.
    Raises QpError(QP_ERR_WORKSPACE) when the cache needs more than STATIC_SCRATCH_BYTES of scratch.
    Calls on one device share that array: do not let two of them overlap on the GPU."""
    _dev_bf16(q)
    if out is None:
        out = torch.empty_like(q)
    st = lib().qp_decode_attn_static(_ptr(q), ctypes.byref(cache.desc), _ptr(out), _stream())
    if st == 4:
        raise QpError(st, f"qp_decode_attn_static: this cache needs more than the built-in "
                          f"{STATIC_SCRATCH_BYTES} bytes of scratch; use qp_decode_attn with a workspace")
    _check(st, "qp_decode_attn_static")
    return out


@dataclass
class Strategy:
    """A quantization strategy of Sec. 5.3 (qp_strategy) with torch-owned side-list buffers."""
    desc: qp_strategy
    bufs: list


def make_strategy(cache: Cache, k_axis: int = 0, outlier_threshold: float | None = None, cap: int | None = None) -> Strategy:
    """Fills a qp_strategy; with filtering on, allocates the two side lists for `cache` (cap entries per
    (batch, KV head), default 4 % of the head's elements)."""
    d = cache.desc
    s = qp_strategy()
    s.k_axis = k_axis
    s.outlier_threshold = float(outlier_threshold) if outlier_threshold else 0.0
    bufs = []
    if outlier_threshold:
        n = d.n_cap or d.n_keep
        cap = cap or max(64, n * d.head_dim // 25)
        dev = cache.k_codes.device
        for side in (s.k_side, s.v_side):
            idx = torch.zeros((d.batch, d.n_kv_heads, cap), dtype=torch.int32, device=dev)
            val = torch.zeros((d.batch, d.n_kv_heads, cap), dtype=torch.bfloat16, device=dev)
            cnt = torch.zeros((d.batch, d.n_kv_heads), dtype=torch.int32, device=dev)
            tp = torch.zeros((d.batch, d.n_kv_heads, (n + 31) // 32 + 1), dtype=torch.int32, device=dev)
            side.cap, side.idx, side.val, side.cnt, side.tile_ptr = cap, _ptr(idx), _ptr(val), _ptr(cnt), _ptr(tp)
            bufs.append((idx, val, cnt, tp))
    return Strategy(s, bufs)


def gather_quantize_ex(K: torch.Tensor, V: torch.Tensor, kept_idx: torch.Tensor, cache: Cache, strategy: Strategy) -> Cache:
    _dev_bf16(K); _dev_bf16(V)
    assert kept_idx.is_cuda and kept_idx.dtype == torch.int32 and kept_idx.is_contiguous()
    _check(lib().qp_gather_quantize_ex(_ptr(K), _ptr(V), _ptr(kept_idx), K.shape[2], ctypes.byref(cache.desc),
                                       ctypes.byref(strategy.desc), _stream()), "qp_gather_quantize_ex")
    return cache


def decode_attn_ex(q: torch.Tensor, cache: Cache, strategy: Strategy, out: torch.Tensor | None = None,
                   workspace: torch.Tensor | None = None) -> torch.Tensor:
    _dev_bf16(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_decode_workspace(decode_workspace_bytes(cache), q.device)
    _check(lib().qp_decode_attn_ex(_ptr(q), ctypes.byref(cache.desc), ctypes.byref(strategy.desc), _ptr(out),
                                   _ptr(workspace), workspace.numel(), _stream()), "qp_decode_attn_ex")
    return out


def decode_attn_layers_ex(qs: list[torch.Tensor], caches: list[Cache], strategy: Strategy, outs: list[torch.Tensor],
                          workspace: torch.Tensor | None = None) -> None:
    n = len(caches)
    assert 1 <= n <= QP_MAX_LAYERS and len(qs) == n and len(outs) == n
    if workspace is None:
        workspace = new_decode_workspace(sum(decode_workspace_bytes(c) for c in caches), qs[0].device)
    arr = lambda ts: (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])
    _check(lib().qp_decode_attn_layers_ex(n, arr(qs), (qp_cache * n)(*[c.desc for c in caches]),
                                          ctypes.byref(strategy.desc), arr(outs), _ptr(workspace), workspace.numel(),
                                          _stream()), "qp_decode_attn_layers_ex")


def head_budgets(scores: torch.Tensor, L: int, w: int, n_mean: int, unit: int = 32) -> torch.Tensor:
    """qp_head_budgets: scores fp32 [Bt,Hkv,P] (device) -> tokens kept per KV head, int32 [Bt,Hkv] (device)."""
    assert scores.is_cuda and scores.dtype == torch.float32 and scores.is_contiguous()
    Bt, Hkv, P = scores.shape
    assert P == L - w
    out = torch.empty((Bt, Hkv), dtype=torch.int32, device=scores.device)
    ws = torch.empty(max(16, int(lib().qp_head_budgets_workspace_bytes(Bt, Hkv, L, w, n_mean))), dtype=torch.uint8,
                     device=scores.device)
    _check(lib().qp_head_budgets(_ptr(scores), Bt, Hkv, L, w, n_mean, unit, _ptr(out), _ptr(ws), ws.numel(), _stream()),
           "qp_head_budgets")
    return out


@dataclass
class HeadCaches:
    """One packed cache per (batch, KV head) of a layer pruned with head-level budgets (descriptors with
    batch = 1, n_kv_heads = 1, n_q_heads = G), in (batch, head) order, and the strategy they were written with."""
    caches: list
    kept: list
    n_heads: list            # tokens kept per (batch, KV head), host ints
    strategy: "Strategy | None"
    shape: tuple             # (Bt, Hq, Hkv, D)


def compress_layer_heads(K: torch.Tensor, V: torch.Tensor, Q_win: torch.Tensor, n_mean: int, bits: int, group: int = 32,
                         pool: int = 7, k_axis: int = 1, unit: int | None = None) -> HeadCaches:
    """The prefill-side path with head-level budgets: qp_window_scores -> qp_head_budgets -> (one copy of the
    Bt x Hkv counts to the host, to size the heads' caches) -> per head qp_select_topk and
    qp_gather_quantize(_ex).  k_axis = 1: keys per token, the arrangement the paper pairs with these methods;
    k_axis = 0: the main path's per-channel keys (unit must then be a multiple of the group)."""
    _dev_bf16(K); _dev_bf16(V); _dev_bf16(Q_win)
    Bt, Hq, Hkv, D, L, w = _dims(K, Q_win)
    G = Hq // Hkv
    unit = unit or group
    scores = window_scores(Q_win, K, pool)
    n_dev = head_budgets(scores, L, w, n_mean, unit)
    n_host = n_dev.cpu().view(-1).tolist()             # the one host round trip of this path
    caches, kepts = [], []
    strategy = None
    for i, n in enumerate(n_host):
        b, h = divmod(i, Hkv)
        c = alloc_cache(1, G, 1, D, bits, group, n, K.device)
        kept = torch.empty((1, 1, n), dtype=torch.int32, device=K.device)
        _check(lib().qp_select_topk(scores[b, h].data_ptr(), 1, 1, L, w, n, _ptr(kept), _stream()), "qp_select_topk")
        if bits == 16 or k_axis == 0:
            _check(lib().qp_gather_quantize(K[b, h].data_ptr(), V[b, h].data_ptr(), _ptr(kept), L, ctypes.byref(c.desc),
                                            _stream()), "qp_gather_quantize")
        else:
            strategy = strategy or make_strategy(c, 1, None)
            _check(lib().qp_gather_quantize_ex(K[b, h].data_ptr(), V[b, h].data_ptr(), _ptr(kept), L, ctypes.byref(c.desc),
                                               ctypes.byref(strategy.desc), _stream()), "qp_gather_quantize_ex")
        caches.append(c); kepts.append(kept)
    return HeadCaches(caches, kepts, n_host, strategy, (Bt, Hq, Hkv, D))


def decode_attn_heads(q: torch.Tensor, hc: HeadCaches, out: torch.Tensor | None = None) -> torch.Tensor:
    """Decode attention over the per-head caches of compress_layer_heads: q, out bf16 [Bt,Hq,D]; every head is one
    entry of a multi-cache call (qp_decode_attn_layers, or qp_decode_attn_layers_ex for per-token keys)."""
    _dev_bf16(q)
    Bt, Hq, Hkv, D = hc.shape
    G = Hq // Hkv
    if out is None:
        out = torch.empty_like(q)
    qv, ov = q.view(Bt * Hkv, 1, G, D), out.view(Bt * Hkv, 1, G, D)
    for lo in range(0, len(hc.caches), QP_MAX_LAYERS):
        hi = min(len(hc.caches), lo + QP_MAX_LAYERS)
        qs, outs = [qv[i] for i in range(lo, hi)], [ov[i] for i in range(lo, hi)]
        if hc.strategy is None:
            decode_attn_layers(LayerBatch(qs, hc.caches[lo:hi], outs))
        else:
            decode_attn_layers_ex(qs, hc.caches[lo:hi], hc.strategy, outs)
    return out


def debug_check() -> tuple[int, list[int]]:
    """qp_debug_check: (status, [1 + site of the first violation or 0, index, limit, violations]); status is
    QP_ERR_UNSUPPORTED (2) unless the loaded library is the range-checked build."""
    w = (ctypes.c_uint32 * 4)()
    st = lib().qp_debug_check(w)
    return st, list(w)


# the C entry points under their own names
qp_status_string = status_string
qp_n_keep = n_keep
qp_cache_layout = cache_layout
qp_compress_workspace_bytes = compress_workspace_bytes
qp_decode_workspace_bytes = decode_workspace_bytes
qp_window_scores = window_scores
qp_select_topk = select_topk
qp_gather_quantize = gather_quantize
qp_compress_layer = compress_layer
qp_compress_layers = compress_layers
qp_decode_attn = decode_attn
qp_decode_attn_layers = decode_attn_layers
qp_decode_attn_static = decode_attn_static
qp_decode_overlap = decode_overlap
qp_gather_quantize_ex = gather_quantize_ex
qp_decode_attn_ex = decode_attn_ex
qp_debug_check = debug_check
qp_decode_attn_layers_ex = decode_attn_layers_ex
qp_head_budgets = head_budgets
qp_head_budgets_workspace_bytes = lambda *a: int(lib().qp_head_budgets_workspace_bytes(*a))
qp_cache_layout_cap = cache_layout_cap
qp_append_kv = append_kv
qp_append_kv_layers = append_kv_layers
qp_decode_attn_tail = decode_attn_tail
qp_decode_attn_tail_layers = decode_attn_tail_layers
