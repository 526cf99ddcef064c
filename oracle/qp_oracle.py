"""ctypes front end of the CPU oracle (``qp_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The GPU library never imports this module and this
module never imports the GPU library.

All arrays are numpy.  bf16 and fp16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qp_oracle.c")
_LIB = os.path.join(_HERE, "libqp_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i, i64, p = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p
        L.qpo_n_keep.restype = i64
        L.qpo_n_keep.argtypes = [i64, i, i, i, i]
        L.qpo_scores.restype = None
        L.qpo_scores.argtypes = [p, p, i, i, i, i, i, i, i, p, p]
        L.qpo_select.restype = None
        L.qpo_select.argtypes = [p, i, i, i, i, i, p]
        L.qpo_quantize.restype = None
        L.qpo_quantize.argtypes = [p, p, p, i, i, i, i, i, i, i, p, p, p, p, p, p]
        L.qpo_dequantize.restype = None
        L.qpo_dequantize.argtypes = [p, p, p, p, p, p, i, i, i, i, i, i, p, p]
        L.qpo_decode.restype = None
        L.qpo_decode.argtypes = [p, p, p, i, i, i, i, i, p]
        L.qpo_quantize_ex.restype = None
        L.qpo_quantize_ex.argtypes = [p, p, p, i, i, i, i, i, i, i, i, ctypes.c_float] + [p] * 12 + [i]
        L.qpo_dequantize_ex.restype = None
        L.qpo_dequantize_ex.argtypes = [p] * 6 + [i] * 7 + [p] * 6 + [i, p, p]
        L.qpo_f32_to_f16_down.restype = ctypes.c_uint16
        L.qpo_f32_to_f16_down.argtypes = [ctypes.c_float]
        L.qpo_f32_to_f16_up.restype = ctypes.c_uint16
        L.qpo_f32_to_f16_up.argtypes = [ctypes.c_float]
        L.qpo_f16_to_f32.restype = ctypes.c_float
        L.qpo_f16_to_f32.argtypes = [ctypes.c_uint16]
        L.qpo_num_threads.restype = i
        L.qpo_num_threads.argtypes = []
        _lib = L
    return _lib


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == dtype, (a.dtype, dtype)
    return a


def num_threads() -> int:
    return int(lib().qpo_num_threads())


def n_keep(budget_bits: int, bits: int, group: int, L: int, w: int) -> int:
    return int(lib().qpo_n_keep(budget_bits, bits, group, L, w))


def f32_to_f16_down(x: float) -> int:
    return int(lib().qpo_f32_to_f16_down(x))


def f32_to_f16_up(x: float) -> int:
    return int(lib().qpo_f32_to_f16_up(x))


def f16_to_f32(h: int) -> float:
    return float(lib().qpo_f16_to_f32(h))


def scores(q_win: np.ndarray, k: np.ndarray, pool: int = 7, want_votes: bool = False):
    """q_win [Bt,Hq,w,D], k [Bt,Hkv,L,D] uint16(bf16) -> pooled [Bt,Hkv,P] fp64."""
    q_win, k = _c(q_win, np.uint16), _c(k, np.uint16)
    Bt, Hq, w, D = q_win.shape
    _, Hkv, L, _ = k.shape
    P = L - w
    pooled = np.empty((Bt, Hkv, P), np.float64)
    votes = np.empty((Bt, Hkv, P), np.float64) if want_votes else None
    lib().qpo_scores(_p(q_win), _p(k), Bt, Hq, Hkv, D, L, w, pool, _p(pooled), _p(votes))
    return (pooled, votes) if want_votes else pooled


def select(pooled: np.ndarray, L: int, w: int, n: int) -> np.ndarray:
    """pooled [Bt,Hkv,P] fp64 -> kept [Bt,Hkv,n] int32 ascending."""
    pooled = _c(pooled, np.float64)
    Bt, Hkv, P = pooled.shape
    assert P == L - w
    kept = np.empty((Bt, Hkv, n), np.int32)
    lib().qpo_select(_p(pooled), Bt, Hkv, L, w, n, _p(kept))
    return kept


@dataclass
class Packed:
    """The packed pruned cache of one layer, in the library's documented layout."""
    bits: int
    group: int
    n: int
    k_codes: np.ndarray   # u32 [Bt,Hkv,n/g,D,wpg]   (bits 16: u16 [Bt,Hkv,n,D])
    v_codes: np.ndarray   # u32 [Bt,Hkv,n,D/g,wpg]   (bits 16: u16 [Bt,Hkv,n,D])
    k_scale: np.ndarray | None  # u16(fp16) [Bt,Hkv,n/g,D]
    k_zero: np.ndarray | None
    v_scale: np.ndarray | None  # u16(fp16) [Bt,Hkv,n,D/g]
    v_zero: np.ndarray | None
    # the other strategies of Sec. 5.3 (qpo_quantize_ex); defaults = the method's own (KIVI axes, no filtering)
    k_axis: int = 0                     # 1: keys grouped per token like the values: k_codes [Bt,Hkv,n,D/g,wpg]
    k_side: "Side | None" = None        # outliers kept in 16 bit, keys / values
    v_side: "Side | None" = None


@dataclass
class Side:
    """Outliers of every (batch, KV head), ascending in t*D + d (t = index among the kept tokens)."""
    idx: np.ndarray    # int32 [Bt,Hkv,cap]
    val: np.ndarray    # u16(bf16) [Bt,Hkv,cap]
    cnt: np.ndarray    # int32 [Bt,Hkv]


def quantize(k: np.ndarray, v: np.ndarray, kept: np.ndarray, bits: int, group: int) -> Packed:
    k, v, kept = _c(k, np.uint16), _c(v, np.uint16), _c(kept, np.int32)
    Bt, Hkv, L, D = k.shape
    n = kept.shape[-1]
    if bits == 16:
        kc = np.empty((Bt, Hkv, n, D), np.uint16)
        vc = np.empty((Bt, Hkv, n, D), np.uint16)
        lib().qpo_quantize(_p(k), _p(v), _p(kept), Bt, Hkv, D, L, n, bits, group,
                           _p(kc), None, None, _p(vc), None, None)
        return Packed(bits, group, n, kc, vc, None, None, None, None)
    assert n % group == 0 and D % group == 0
    wpg = group * bits // 32
    kc = np.empty((Bt, Hkv, n // group, D, wpg), np.uint32)
    ks = np.empty((Bt, Hkv, n // group, D), np.uint16)
    kz = np.empty_like(ks)
    vc = np.empty((Bt, Hkv, n, D // group, wpg), np.uint32)
    vs = np.empty((Bt, Hkv, n, D // group), np.uint16)
    vz = np.empty_like(vs)
    lib().qpo_quantize(_p(k), _p(v), _p(kept), Bt, Hkv, D, L, n, bits, group,
                       _p(kc), _p(ks), _p(kz), _p(vc), _p(vs), _p(vz))
    return Packed(bits, group, n, kc, vc, ks, kz, vs, vz)


def quantize_ex(k: np.ndarray, v: np.ndarray, kept: np.ndarray, bits: int, group: int, k_axis: int = 0,
                outlier_threshold: float | None = None, cap: int | None = None) -> Packed:
    """The quantization strategies of Sec. 5.3: key grouping axis and outlier filtering (bits < 16)."""
    k, v, kept = _c(k, np.uint16), _c(v, np.uint16), _c(kept, np.int32)
    Bt, Hkv, L, D = k.shape
    n = kept.shape[-1]
    assert bits < 16 and D % group == 0 and (k_axis == 1 or n % group == 0)
    wpg = group * bits // 32
    if k_axis == 0:
        kc = np.empty((Bt, Hkv, n // group, D, wpg), np.uint32)
        ks = np.empty((Bt, Hkv, n // group, D), np.uint16)
    else:
        kc = np.empty((Bt, Hkv, n, D // group, wpg), np.uint32)
        ks = np.empty((Bt, Hkv, n, D // group), np.uint16)
    kz = np.empty_like(ks)
    vc = np.empty((Bt, Hkv, n, D // group, wpg), np.uint32)
    vs = np.empty((Bt, Hkv, n, D // group), np.uint16)
    vz = np.empty_like(vs)
    filt = outlier_threshold is not None
    cap = (n * D if cap is None else cap) if filt else 1
    sides = [Side(np.zeros((Bt, Hkv, cap), np.int32), np.zeros((Bt, Hkv, cap), np.uint16),
                  np.zeros((Bt, Hkv), np.int32)) for _ in range(2)]
    lib().qpo_quantize_ex(_p(k), _p(v), _p(kept), Bt, Hkv, D, L, n, bits, group, k_axis,
                          float(outlier_threshold) if filt else float("inf"),
                          _p(kc), _p(ks), _p(kz), _p(vc), _p(vs), _p(vz),
                          _p(sides[0].idx), _p(sides[0].val), _p(sides[0].cnt),
                          _p(sides[1].idx), _p(sides[1].val), _p(sides[1].cnt), cap)
    return Packed(bits, group, n, kc, vc, ks, kz, vs, vz, k_axis, sides[0] if filt else None,
                  sides[1] if filt else None)


def dequantize(pk: Packed, D: int):
    """-> (K', V') fp64 [Bt,Hkv,n,D]  (Eq. 5)."""
    Bt, Hkv = pk.k_codes.shape[:2]
    kd = np.empty((Bt, Hkv, pk.n, D), np.float64)
    vd = np.empty_like(kd)
    if pk.k_axis != 0 or pk.k_side is not None:
        ksd, vsd = pk.k_side, pk.v_side
        cap = ksd.idx.shape[-1] if ksd is not None else 1
        lib().qpo_dequantize_ex(_p(pk.k_codes), _p(pk.k_scale), _p(pk.k_zero), _p(pk.v_codes), _p(pk.v_scale),
                                _p(pk.v_zero), Bt, Hkv, D, pk.n, pk.bits, pk.group, pk.k_axis,
                                _p(ksd.idx) if ksd else None, _p(ksd.val) if ksd else None,
                                _p(ksd.cnt) if ksd else None, _p(vsd.idx) if vsd else None,
                                _p(vsd.val) if vsd else None, _p(vsd.cnt) if vsd else None, cap, _p(kd), _p(vd))
        return kd, vd
    lib().qpo_dequantize(_p(pk.k_codes), _p(pk.k_scale), _p(pk.k_zero), _p(pk.v_codes),
                         _p(pk.v_scale), _p(pk.v_zero), Bt, Hkv, D, pk.n, pk.bits, pk.group,
                         _p(kd), _p(vd))
    return kd, vd


def decode(q: np.ndarray, kd: np.ndarray, vd: np.ndarray) -> np.ndarray:
    """q [Bt,Hq,D] uint16(bf16); kd, vd fp64 [Bt,Hkv,n,D] -> out fp64 [Bt,Hq,D]  (Eq. 3)."""
    q, kd, vd = _c(q, np.uint16), _c(kd, np.float64), _c(vd, np.float64)
    Bt, Hq, D = q.shape
    _, Hkv, n, _ = kd.shape
    out = np.empty((Bt, Hq, D), np.float64)
    lib().qpo_decode(_p(q), _p(kd), _p(vd), Bt, Hq, Hkv, D, n, _p(out))
    return out


def compress_layer(k, v, q_win, budget_bits: int, bits: int, group: int = 32, pool: int = 7):
    """The whole prefill-side path on the CPU: scores -> select -> gather+quantize."""
    L, w = k.shape[2], q_win.shape[2]
    n = n_keep(budget_bits, bits, group, L, w)
    if n < 0:
        raise ValueError("budget cannot be met")
    pooled = scores(q_win, k, pool)
    kept = select(pooled, L, w, n)
    return quantize(k, v, kept, bits, group), kept, pooled


# ------------------------------------------------------------------ decode-time appends (Eq. 2)

@dataclass
class GenState:
    """Cache of one layer during generation: the packed part plus a 16-bit tail.

    Eq. 2 appends the new token's key and value to the cache.  The paper does not say how a
    quantized cache takes in single tokens, and key groups span g tokens, so the reading here is:
    appended tokens wait, unquantized (bf16), in a tail of fewer than g tokens per KV head;
    attention runs over the packed tokens followed by the tail; as soon as the tail holds g tokens
    they are quantized by Eq. 4 exactly like g kept tokens of the prompt (one key group per channel,
    g value rows) and become the last g tokens of the packed part.  At 16 bit nothing waits: the
    row goes straight into the cache.  Nothing is pruned after the prompt.
    """
    packed: Packed
    tail_k: np.ndarray   # u16(bf16) [Bt,Hkv,n_tail,D], 0 <= n_tail < g
    tail_v: np.ndarray

    @property
    def n_tail(self) -> int:
        return self.tail_k.shape[2]


def gen_state(pk: Packed, D: int) -> GenState:
    Bt, Hkv = pk.k_codes.shape[:2]
    e = np.empty((Bt, Hkv, 0, D), np.uint16)
    return GenState(pk, e, e.copy())


def _concat_packed(a: Packed, b: Packed) -> Packed:
    """The tokens of b after the tokens of a (every array of the layout has its token or
    token-group axis third)."""
    cat = lambda x, y: None if x is None else np.concatenate([x, y], axis=2)
    return Packed(a.bits, a.group, a.n + b.n, cat(a.k_codes, b.k_codes), cat(a.v_codes, b.v_codes),
                  cat(a.k_scale, b.k_scale), cat(a.k_zero, b.k_zero),
                  cat(a.v_scale, b.v_scale), cat(a.v_zero, b.v_zero))


def append(st: GenState, k_new: np.ndarray, v_new: np.ndarray) -> GenState:
    """k_new, v_new u16(bf16) [Bt,Hkv,D]: the new token's key and value rows (Eq. 2)."""
    k_new, v_new = _c(k_new, np.uint16), _c(v_new, np.uint16)
    tk = np.concatenate([st.tail_k, k_new[:, :, None, :]], axis=2)
    tv = np.concatenate([st.tail_v, v_new[:, :, None, :]], axis=2)
    pk = st.packed
    full = 1 if pk.bits == 16 else pk.group
    if tk.shape[2] < full:
        return GenState(pk, tk, tv)
    Bt, Hkv, _, D = tk.shape
    ident = np.broadcast_to(np.arange(full, dtype=np.int32), (Bt, Hkv, full)).copy()
    flushed = quantize(tk, tv, ident, pk.bits, pk.group)
    return GenState(_concat_packed(pk, flushed), tk[:, :, :0].copy(), tv[:, :, :0].copy())


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def decode_state(q: np.ndarray, st: GenState, D: int) -> np.ndarray:
    """Eq. 3 over the dequantized packed tokens (Eq. 5) followed by the tail's exact values."""
    kd, vd = dequantize(st.packed, D)
    if st.n_tail:
        kd = np.concatenate([kd, _bf16_to_f64(st.tail_k)], axis=2)
        vd = np.concatenate([vd, _bf16_to_f64(st.tail_v)], axis=2)
    return decode(q, kd, vd)


# ------------------------------------------------------------------ head-level token budgets

def head_budgets(pooled: np.ndarray, L: int, w: int, n_mean: int, unit: int = 32) -> np.ndarray:
    """Tokens kept per KV head when the layer's budget is shared between its heads.

    The paper runs two pruning methods of this kind (Ada-KV, HeadKV: Related Work "KV Pruning", Sec. 4
    "Setup", Table 1) and only says of them that they retain different numbers of tokens per head.  The rule
    taken here: within one batch entry the Hkv * (n_mean - w) prefix positions with the largest pooled scores
    over ALL KV heads are marked (equal scores: lower head first, then lower position); a head's raw share is
    its number of marked positions plus its w window tokens.  Shares are rounded down to whole units of
    `unit` tokens, raised to the smallest whole unit count above w where they fall below it, capped at L
    rounded down to units, and, should the raising have pushed the total above Hkv * n_mean, the largest heads
    (lowest head first among equals) give back one unit at a time.  pooled [Bt,Hkv,P] -> n [Bt,Hkv] int32.
    """
    pooled = np.asarray(pooled, np.float64)
    Bt, Hkv, P = pooled.shape
    assert P == L - w and n_mean > w
    k_total = min(Hkv * (n_mean - w), Hkv * P)
    floor_u = lambda x: (x // unit) * unit
    n_min = floor_u(w) + unit                          # smallest whole number of units above w
    n_max = max(n_min, floor_u(L))
    out = np.zeros((Bt, Hkv), np.int32)
    for b in range(Bt):
        items = [(-pooled[b, h, j], h, j) for h in range(Hkv) for j in range(P)]
        items.sort()
        raw = [w] * Hkv
        for _, h, _j in items[:k_total]:
            raw[h] += 1
        n = [min(n_max, max(n_min, floor_u(r))) for r in raw]
        while sum(n) > Hkv * n_mean and max(n) > n_min:
            h = max(range(Hkv), key=lambda i: (n[i], -i))
            n[h] -= unit
        out[b] = n
    return out
