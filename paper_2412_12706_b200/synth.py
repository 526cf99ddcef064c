"""Seeded synthetic inputs: shapes and value structure of Llama-3-class KV caches.

This module only produces *inputs* (K, V, window queries, decode queries).  It
contains none of the method's arithmetic and imports neither the GPU library nor
the CPU oracle; both are fed from here.

Generator: counter based.  Element ``i`` of tensor ``tid`` of layer ``layer`` is a
function of ``(seed, layer, tid, i)`` only, so any slice can be regenerated
anywhere.  A 64-bit integer mixer (the splitmix64 finaliser) yields three words
per element = twelve 16-bit uniforms; their sum, centred and divided by 65536,
is an Irwin-Hall normal variate (mean 0, std 1, |x| < 6).  All of it is integer
arithmetic followed by one exact power-of-two scaling, so CPU and CUDA devices
give the same bits.  The result is rounded to bf16 (round to nearest even).
"""
from __future__ import annotations

import dataclasses
import math

import torch

BASE_SEED = 20241217

_M1 = 0xBF58476D1CE4E5B9 - (1 << 64)   # as signed 64-bit
_M2 = 0x94D049BB133111EB - (1 << 64)
_GOLD = 0x9E3779B97F4A7C15 - (1 << 64)
_MASK16 = 0xFFFF


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _M1
    x = (x ^ _lsr(x, 27)) * _M2
    return x ^ _lsr(x, 31)


def _key(seed: int, layer: int, tid: int) -> int:
    """Scalar stream key (Python ints, wrapped to signed 64-bit)."""
    def mix1(v: int) -> int:
        v &= (1 << 64) - 1
        v = ((v ^ (v >> 30)) * 0xBF58476D1CE4E5B9) & ((1 << 64) - 1)
        v = ((v ^ (v >> 27)) * 0x94D049BB133111EB) & ((1 << 64) - 1)
        return v ^ (v >> 31)
    k = mix1(seed * 0x9E3779B97F4A7C15 + 1)
    k = mix1(k ^ (layer * 0xD1B54A32D192ED03 + 2))
    k = mix1(k ^ (tid * 0x8CB92BA72F3D8DD7 + 3))
    return k - (1 << 64) if k >= (1 << 63) else k


def normal_f32(seed: int, layer: int, tid: int, numel: int, device="cpu", offset: int = 0,
               chunk: int = 1 << 24) -> torch.Tensor:
    """Elements ``offset .. offset+numel`` of stream ``(seed, layer, tid)``: Irwin-Hall(12)
    normal variates as exact fp32 (flat tensor)."""
    key = _key(seed, layer, tid)
    out = torch.empty(numel, dtype=torch.float32, device=device)
    for lo in range(0, numel, chunk):
        hi = min(numel, lo + chunk)
        ctr = (torch.arange(lo, hi, dtype=torch.int64, device=device) + offset) * 3
        acc = torch.zeros(hi - lo, dtype=torch.int64, device=device)
        for r in range(3):
            wds = _mix((ctr + r) * _GOLD + key)
            acc += (wds & _MASK16) + (_lsr(wds, 16) & _MASK16) + (_lsr(wds, 32) & _MASK16) \
                + (_lsr(wds, 48) & _MASK16)
        out[lo:hi] = (acc - 393210).to(torch.float32) * (1.0 / 65536.0)
    return out


def _bf16(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.bfloat16)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration (names follow the paper's notation)."""
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    L: int                   # context (prompt) length
    w: int                   # observation window
    tokens16: int            # budget in tokens at 16-bit; budget_bits = 16 * tokens16
    bits: int
    group: int = 32
    pool: int = 7
    decode_steps: int = 16
    structure: str = "outlier"   # "outlier" | "rotary"
    outlier_channels: int = 3
    outlier_scale: float = 8.0
    seed: int = BASE_SEED
    pyramid: bool = False        # per-layer budgets falling linearly from 2x to 0.5x of the mean

    @property
    def budget_bits(self) -> int:
        return 16 * self.tokens16

    def n_keep(self, layer: int = 0) -> int:
        n = self.budget_bits // self.bits
        if self.pyramid:
            frac = 2.0 - 1.5 * layer / max(1, self.n_layers - 1)
            n = int(math.floor(n * frac / 32.0)) * 32
        return min(n, self.L)

    def layer_budget_bits(self, layer: int = 0) -> int:
        return self.n_keep(layer) * self.bits


# The five configurations of the benchmark contract.
TINY = Workload("tiny", 1, 1, 8, 2, 64, 1024, 32, 128, 4, decode_steps=16,
                outlier_channels=4, outlier_scale=10.0, seed=BASE_SEED + 0)
LLAMA8B_8K = Workload("llama3-8b-8k-b1-4bit", 32, 1, 32, 8, 128, 8192, 32, 512, 4,
                      decode_steps=128, seed=BASE_SEED + 1)
LLAMA8B_32K_B8 = Workload("llama3-8b-32k-b8-2bit", 32, 8, 32, 8, 128, 32768, 32, 1024, 2,
                          decode_steps=256, structure="rotary", seed=BASE_SEED + 2)


def sweep_128k(bits: int) -> Workload:
    return Workload(f"llama3-8b-128k-b1-{bits}bit", 32, 1, 32, 8, 128, 131072, 64, 1024, bits,
                    decode_steps=256, seed=BASE_SEED + 3)


LLAMA70B_32K_B4 = Workload("llama3-70b-32k-b4-4bit-pyramid", 80, 4, 64, 8, 128, 32768, 32, 1024, 4,
                           decode_steps=512, seed=BASE_SEED + 4, pyramid=True)

WORKLOADS = {w.name: w for w in (TINY, LLAMA8B_8K, LLAMA8B_32K_B8, sweep_128k(16), sweep_128k(8),
                                 sweep_128k(4), sweep_128k(2), LLAMA70B_32K_B4)}

_TID_K, _TID_V, _TID_QWIN, _TID_QDEC, _TID_PHASE, _TID_KNEW, _TID_VNEW = 1, 2, 3, 4, 5, 6, 7


def _outlier_channels(wl: Workload, hk: int) -> list[int]:
    """Fixed per-KV-head set of key channels that carry large magnitudes."""
    chans: list[int] = []
    c = 0
    while len(chans) < wl.outlier_channels:
        d = (_key(wl.seed, hk, 1000 + c) & 0x7FFFFFFF) % wl.head_dim
        c += 1
        if d not in chans:
            chans.append(d)
    return chans


def make_kv(wl: Workload, layer: int, device="cpu", batch_slice: slice | None = None):
    """K, V [Bt,Hkv,L,D] bf16 for one layer (optionally only some batch entries)."""
    Bt, Hkv, L, D = wl.batch, wl.n_kv_heads, wl.L, wl.head_dim
    per_b = Hkv * L * D
    b0, b1 = (0, Bt) if batch_slice is None else (batch_slice.start or 0, batch_slice.stop or Bt)
    nb = b1 - b0

    def block(tid):
        # exactly the elements [b0*per_b, b1*per_b) of the full tensor
        return normal_f32(wl.seed, layer, tid, nb * per_b, device, offset=b0 * per_b) \
            .view(nb, Hkv, L, D)

    k = block(_TID_K)
    v = block(_TID_V)
    if wl.structure == "outlier":
        for hk in range(Hkv):
            for d in _outlier_channels(wl, hk):
                k[:, hk, :, d] *= wl.outlier_scale
    elif wl.structure == "rotary":
        # K[t,d] = A*sin(t*theta_d + phi_{h,d}) + sigma*N(0,1); channel pairs share a frequency
        A, sigma, base = 2.0, 1.0, 10000.0
        t = torch.arange(L, dtype=torch.float64)
        pair = torch.arange(D, dtype=torch.float64) // 2
        theta = base ** (-2.0 * pair / D)
        quarter = (torch.arange(D) % 2).to(torch.float64) * (math.pi / 2)   # sin / cos pair
        ph = normal_f32(wl.seed, layer, _TID_PHASE, Hkv * D).to(torch.float64).view(Hkv, D) * math.pi
        wave = torch.sin(t[None, :, None] * theta[None, None, :] + quarter[None, None, :]
                         + ph[:, None, :])                                   # [Hkv,L,D] fp64 on CPU
        k = k * sigma + (A * wave).to(torch.float32).to(device)[None]
    else:
        raise ValueError(wl.structure)
    return _bf16(k), _bf16(v)


def make_q_win(wl: Workload, layer: int, device="cpu") -> torch.Tensor:
    """Window queries [Bt,Hq,w,D] bf16 (the last w prompt positions, post-RoPE)."""
    n = wl.batch * wl.n_q_heads * wl.w * wl.head_dim
    return _bf16(normal_f32(wl.seed, layer, _TID_QWIN, n, device)
                 .view(wl.batch, wl.n_q_heads, wl.w, wl.head_dim))


def make_q_dec(wl: Workload, layer: int, step: int, device="cpu") -> torch.Tensor:
    """Decode query [Bt,Hq,D] bf16 of one decode step."""
    n = wl.batch * wl.n_q_heads * wl.head_dim
    return _bf16(normal_f32(wl.seed, layer, _TID_QDEC + 16 * (step + 1), n, device)
                 .view(wl.batch, wl.n_q_heads, wl.head_dim))


def make_kv_new(wl: Workload, layer: int, step: int, device="cpu"):
    """Key and value rows [Bt,Hkv,D] bf16 of the token generated at decode step `step` (same value
    structure as the prompt's keys: the per-head outlier channels stay outliers)."""
    Bt, Hkv, D = wl.batch, wl.n_kv_heads, wl.head_dim
    n = Bt * Hkv * D
    k = normal_f32(wl.seed, layer, _TID_KNEW + 16 * (step + 1), n, device).view(Bt, Hkv, D)
    v = normal_f32(wl.seed, layer, _TID_VNEW + 16 * (step + 1), n, device).view(Bt, Hkv, D)
    if wl.structure == "outlier":
        for hk in range(Hkv):
            for d in _outlier_channels(wl, hk):
                k[:, hk, d] *= wl.outlier_scale
    return _bf16(k), _bf16(v)


def bits_u16(x: torch.Tensor):
    """bf16/fp16 tensor -> numpy uint16 bit patterns (CPU)."""
    return x.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
