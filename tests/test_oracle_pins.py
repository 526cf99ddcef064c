"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of the expected values below is produced by the oracle itself or by the CUDA
path: they are closed forms, brute force, numpy's own float16 / matmul, or values
the paper prints (tests/golden).
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import qp_oracle as orc

RNG = np.random.default_rng(20241217)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32/fp64 array -> bf16 bit patterns (round to nearest even, via torch)."""
    t = torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_val(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f16_val(bits: np.ndarray) -> np.ndarray:
    return bits.view(np.float16).astype(np.float64)


def unpack(words: np.ndarray, bits: int, g: int) -> np.ndarray:
    """[..., wpg] u32 -> [..., g] codes; independent of the oracle's packer."""
    per = 32 // bits
    e = np.arange(g)
    return (words[..., e // per] >> ((e % per) * bits).astype(np.uint32)) & np.uint32((1 << bits) - 1)


# ----------------------------------------------------------------------------- fp16 conversion

def test_fp16_directed_rounding_matches_numpy_float16():
    xs = np.concatenate([
        RNG.standard_normal(20000).astype(np.float32) * 10,
        (RNG.standard_normal(5000) * 1e-5).astype(np.float32),       # fp16 subnormal range
        (RNG.standard_normal(2000) * 1e-9).astype(np.float32),       # below the smallest subnormal
        np.array([0.0, -0.0, 1.0, -1.0, 65504.0, -65504.0, 65503.9, 6.1e-5, -6.1e-5, 5.96e-8,
                  2.0 ** -24, 2.0 ** -25, -(2.0 ** -25), 0.333333, 1e-40], np.float32)])
    for x in xs:
        near = np.float16(x)
        down = near if float(near) <= float(x) else np.nextafter(near, np.float16(-np.inf))
        up = near if float(near) >= float(x) else np.nextafter(near, np.float16(np.inf))
        got_d = np.uint16(orc.f32_to_f16_down(float(x))).view(np.float16)
        got_u = np.uint16(orc.f32_to_f16_up(float(x))).view(np.float16)
        assert float(got_d) == float(down), (x, got_d, down)
        assert float(got_u) == float(up), (x, got_u, up)
        assert float(got_d) <= float(x) <= float(got_u)


def test_fp16_to_fp32_all_finite_patterns():
    bits = np.arange(0, 1 << 16, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    for b in bits[::7]:
        r = ref[b]
        if np.isfinite(r):
            assert orc.f16_to_f32(int(b)) == float(r)


# ----------------------------------------------------------------------------- budget

def test_budget_triples_from_paper():
    path = os.path.join(os.path.dirname(__file__), "golden", "budget_triples.txt")
    rows = [list(map(int, l.split())) for l in open(path) if l.strip() and not l.startswith("#")]
    budgets = set()
    for full_tokens, full_bits, denom, tokens, bits in rows:
        budget_bits = full_tokens * full_bits // denom       # per (KV head, channel) token-bits
        budgets.add(budget_bits)
        n = orc.n_keep(budget_bits, bits, 32, full_tokens, 32)
        assert n == tokens
        assert n * bits == budget_bits
    assert budgets == {8192}


def test_budget_rejections_and_cap():
    assert orc.n_keep(16 * 128, 4, 32, 1024, 32) == 512
    assert orc.n_keep(16 * 128, 3, 32, 1024, 32) == -1          # unsupported bit width
    assert orc.n_keep(16 * 2, 16, 32, 1024, 32) == -1           # n <= w
    assert orc.n_keep(4 * 40, 4, 32, 1024, 8) == -1             # 40 tokens: not whole groups
    assert orc.n_keep(16 * 5000, 16, 32, 1024, 32) == 1024      # capped at L (keep all)


# ----------------------------------------------------------------------------- S1 scores

def _scores(qw, k, pool=7):
    return orc.scores(bf16_bits(qw), bf16_bits(k), pool, want_votes=True)


def test_scores_zero_queries_closed_form():
    Bt, Hq, Hkv, D, L, w = 2, 4, 2, 64, 96, 8
    G, P = Hq // Hkv, L - w
    k = RNG.standard_normal((Bt, Hkv, L, D))
    pooled, votes = _scores(np.zeros((Bt, Hq, w, D)), k)
    u = G * sum(1.0 / (P + i + 1) for i in range(w))      # every row uniform over its P+i+1 keys
    assert np.allclose(votes, u, rtol=1e-13, atol=0)
    assert np.allclose(pooled[..., 3:P - 3], u, rtol=1e-13)
    for e, f in ((0, 4 / 7), (1, 5 / 7), (2, 6 / 7)):       # zero padding, divisor 7
        assert np.allclose(pooled[..., e], u * f, rtol=1e-13)
        assert np.allclose(pooled[..., P - 1 - e], u * f, rtol=1e-13)


def test_scores_single_spike_closed_form_scaling_gqa_and_causality():
    Bt, Hq, Hkv, D, L, w = 1, 4, 2, 64, 80, 8
    G, P = Hq // Hkv, L - w
    alpha = np.array([1.0, 2.0, 3.0, -1.5])          # per query head, bf16-exact
    beta, jstar, jwin = 4.0, 17, P + 2                 # prefix spike and a spike inside the window
    qw = np.zeros((Bt, Hq, w, D))
    qw[0, :, :, 5] = alpha[:, None]
    k = np.zeros((Bt, Hkv, L, D))
    k[0, :, jstar, 5] = beta
    k[0, :, jwin, 5] = 2 * beta
    pooled, votes = _scores(qw, k, pool=1)
    assert np.array_equal(pooled, votes)               # pool = 1 is the identity
    for hk in range(Hkv):
        exp_star = 0.0
        exp_other = 0.0
        for h in range(hk * G, (hk + 1) * G):
            x1 = alpha[h] * beta / math.sqrt(D)
            x2 = alpha[h] * 2 * beta / math.sqrt(D)
            for i in range(w):
                nvis = P + i + 1
                sees_win = (P + i) >= jwin
                Z = (nvis - 1 - (1 if sees_win else 0)) + math.exp(x1) + (math.exp(x2) if sees_win else 0.0)
                exp_star += math.exp(x1) / Z
                exp_other += 1.0 / Z
        assert votes[0, hk, jstar] == pytest.approx(exp_star, rel=1e-12)
        assert votes[0, hk, 3] == pytest.approx(exp_other, rel=1e-12)
        assert votes[0, hk, P - 1] == pytest.approx(exp_other, rel=1e-12)


def test_scores_match_numpy_dense_softmax():
    Bt, Hq, Hkv, D, L, w = 2, 6, 2, 32, 70, 5
    G, P = Hq // Hkv, L - w
    qb = bf16_bits(RNG.standard_normal((Bt, Hq, w, D)))
    kb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)) * 1.5)
    pooled, votes = orc.scores(qb, kb, 7, want_votes=True)
    q, k = bf16_val(qb), bf16_val(kb)
    for b in range(Bt):
        for hk in range(Hkv):
            vote = np.zeros(P)
            for h in range(hk * G, (hk + 1) * G):
                S = q[b, h] @ k[b, hk].T / math.sqrt(D)              # [w, L]
                mask = np.arange(L)[None, :] > (P + np.arange(w))[:, None]
                S = np.where(mask, -np.inf, S)
                Pm = np.exp(S - S.max(1, keepdims=True))
                Pm /= Pm.sum(1, keepdims=True)
                vote += Pm[:, :P].sum(0)
            assert np.allclose(votes[b, hk], vote, rtol=1e-12)
            ref = np.convolve(vote, np.ones(7), mode="same") / 7
            assert np.allclose(pooled[b, hk], ref, rtol=1e-12)
    # total probability mass: prefix votes + window mass = G*w
    assert np.all(votes.sum(-1) < G * w)


# ----------------------------------------------------------------------------- S2 selection

def test_select_uniform_votes_picks_3_to_k_plus_2():
    # identical key rows -> uniform votes; the pooled score is lower at the 3 edge positions,
    # so the selected prefix set is {3, .., k+2}: pins zero padding, divisor and lowest-index ties
    Bt, Hq, Hkv, D, L, w, n = 1, 2, 1, 32, 72, 8, 32
    P, kk = L - w, n - w
    row = RNG.standard_normal(D)
    k = np.broadcast_to(row, (Bt, Hkv, L, D)).copy()
    qw = RNG.standard_normal((Bt, Hq, w, D))
    pooled = orc.scores(bf16_bits(qw), bf16_bits(k), 7)
    kept = orc.select(pooled, L, w, n)
    assert kept[0, 0, :kk].tolist() == list(range(3, kk + 3))
    assert kept[0, 0, kk:].tolist() == list(range(P, L))


def test_select_spike_keeps_pooled_neighbours():
    Bt, Hq, Hkv, D, L, w, n = 1, 2, 1, 32, 200, 8, 8 + 7
    P = L - w
    qdir = np.zeros(D); qdir[3] = 1.0
    qw = np.broadcast_to(8.0 * qdir, (Bt, Hq, w, D)).copy()
    k = RNG.standard_normal((Bt, Hkv, L, D)) * 0.01
    k[0, 0, 100] = 16.0 * qdir
    pooled = orc.scores(bf16_bits(qw), bf16_bits(k), 7)
    kept = orc.select(pooled, L, w, n)
    assert kept[0, 0, :7].tolist() == list(range(97, 104))


def test_select_brute_force_with_duplicates():
    for trial in range(20):
        Bt, Hkv, L, w = 2, 3, 64 + trial, 4 + trial % 5
        P = L - w
        pooled = RNG.integers(0, 9, size=(Bt, Hkv, P)).astype(np.float64) / 8.0   # many ties
        n = w + 1 + (trial * 3) % (P - 1)
        kept = orc.select(pooled, L, w, n)
        kk = n - w
        for b in range(Bt):
            for h in range(Hkv):
                s = pooled[b, h].copy()
                chosen = []
                for _ in range(kk):                       # repeated argmax; argmax returns lowest index
                    j = int(np.argmax(s))
                    chosen.append(j)
                    s[j] = -1.0
                out = kept[b, h]
                assert out[:kk].tolist() == sorted(chosen)
                assert out[kk:].tolist() == list(range(P, L))
                assert np.all(np.diff(out) > 0)


def test_select_keep_all():
    pooled = RNG.random((1, 1, 24))
    kept = orc.select(pooled, 32, 8, 32)
    assert kept[0, 0].tolist() == list(range(32))


# ----------------------------------------------------------------------------- S3 quantizer

def _quant(k, v, bits, g, kept=None):
    kb, vb = bf16_bits(k), bf16_bits(v)
    Bt, Hkv, L, D = kb.shape
    if kept is None:
        kept = np.broadcast_to(np.arange(L, dtype=np.int32), (Bt, Hkv, L)).copy()
    return orc.quantize(kb, vb, kept, bits, g), kb, vb, kept


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("g", [32, 64])
def test_quantizer_error_bound_and_code_range(bits, g):
    Bt, Hkv, L, D = 1, 2, 128, 64
    k = RNG.standard_normal((Bt, Hkv, L, D)); k[..., 7] *= 10
    v = RNG.standard_normal((Bt, Hkv, L, D))
    pk, kb, vb, _ = _quant(k, v, bits, g)
    kd, vd = orc.dequantize(pk, D)
    kc = unpack(pk.k_codes, bits, g)                    # [Bt,Hkv,n/g,D,g]
    vc = unpack(pk.v_codes, bits, g)                    # [Bt,Hkv,n,D/g,g]
    assert kc.max() <= (1 << bits) - 1 and vc.max() <= (1 << bits) - 1
    ks = f16_val(pk.k_scale)[:, :, :, None, :].repeat(g, 3).reshape(Bt, Hkv, L, D)
    vs = f16_val(pk.v_scale)[..., None].repeat(g, -1).reshape(Bt, Hkv, L, D)
    assert np.all(np.abs(kd - bf16_val(kb)) <= ks / 2 * (1 + 1e-3))
    assert np.all(np.abs(vd - bf16_val(vb)) <= vs / 2 * (1 + 1e-3))
    # every group reaches code 0 at its minimum and the top code at its maximum
    assert np.all(kc.min(-1) == 0) and np.all(kc.max(-1) == (1 << bits) - 1)
    assert np.all(vc.min(-1) == 0) and np.all(vc.max(-1) == (1 << bits) - 1)
    # zero <= group min (rounded down), and min reconstructs with error < one fp16 ulp
    kmin = bf16_val(kb).reshape(Bt, Hkv, L // g, g, D).min(3)
    assert np.all(f16_val(pk.k_zero) <= kmin)


# The three tests below pin the stored-precision rules of one quantization group (Eq. 4 with
# the scale and the zero point held in fp16): each fails if the oracle rounds the scale down or
# to nearest, rounds the zero point up or to nearest, or breaks rounding ties away from zero.

def _group_views(kb, vb, g):
    """bf16 bit arrays [Bt,Hkv,L,D] -> float64 values per group, last axis = the group's elements:
    keys [Bt,Hkv,L/g,D,g] (per channel over g tokens), values [Bt,Hkv,L,D/g,g] (per token)."""
    Bt, Hkv, L, D = kb.shape
    kg = bf16_val(kb).reshape(Bt, Hkv, L // g, g, D).transpose(0, 1, 2, 4, 3)
    vg = bf16_val(vb).reshape(Bt, Hkv, L, D // g, g)
    return kg, vg


def _f16_floor(x: np.ndarray) -> np.ndarray:
    """largest fp16 <= x (x float64), from numpy's own float16 rounding and nextafter"""
    near = x.astype(np.float16)
    lower = np.nextafter(near, np.float16(-np.inf))
    return np.where(near.astype(np.float64) <= x, near, lower)


def _f16_ceil(x: np.ndarray) -> np.ndarray:
    near = x.astype(np.float16)
    upper = np.nextafter(near, np.float16(np.inf))
    return np.where(near.astype(np.float64) >= x, near, upper)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_stored_scale_is_smallest_fp16_not_below_the_exact_quotient(bits):
    g, D, L = 32, 64, 256
    k = RNG.standard_normal((1, 2, L, D)) * 3.0
    v = RNG.standard_normal((1, 2, L, D))
    pk, kb, vb, _ = _quant(k, v, bits, g)
    kg, vg = _group_views(kb, vb, g)
    qmax = (1 << bits) - 1
    checked = 0
    for vals, scale, zero in ((kg, pk.k_scale, pk.k_zero), (vg, pk.v_scale, pk.v_zero)):
        quot = (vals.max(-1) - f16_val(zero)) / qmax          # float64, from the STORED zero point
        want = _f16_ceil(quot)
        got = scale.view(np.float16)
        # a quotient within fp32 rounding of an fp16 value may legitimately land on either side
        gap = np.abs(quot - want.astype(np.float64))
        clear = (gap == 0) | (gap > 4e-7 * quot)          # exactly representable quotients are clear too
        checked += int(clear.sum())
        assert np.array_equal(got[clear], want[clear])
        # never below the quotient (beyond fp32 rounding): the top element must not clip
        assert np.all(got.astype(np.float64) >= quot * (1 - 2e-7))
        # and strictly above it somewhere by a good part of an fp16 step: not round-to-nearest
        assert np.any(got.astype(np.float64) > quot * (1 + 6e-4))
    assert checked > 0.99 * (kg.shape[:-1][2] * kg.shape[3] * 2 + vg.shape[2] * vg.shape[3] * 2)


@pytest.mark.parametrize("magnitude", [1e-6, 1e-7, 1e-9])
def test_stored_zero_is_largest_fp16_not_above_the_minimum(magnitude):
    # minima in and below the fp16 subnormal range (spacing 2^-24 = 6e-8): bf16 holds them
    # exactly, fp16 does not, so the direction of the zero point's rounding shows
    bits, g, D, L = 4, 32, 32, 64
    k = RNG.standard_normal((1, 1, L, D)) * magnitude
    v = RNG.standard_normal((1, 1, L, D)) * magnitude
    k[0, 0, :, 0] = np.abs(k[0, 0, :, 0]) + magnitude        # an all-positive group: zero must not exceed min
    pk, kb, vb, _ = _quant(k, v, bits, g)
    kg, vg = _group_views(kb, vb, g)
    inexact = 0
    for vals, zero in ((kg, pk.k_zero), (vg, pk.v_zero)):
        mn = vals.min(-1)
        want = _f16_floor(mn)
        got = zero.view(np.float16)
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16))     # bit patterns: -0.0 vs 0.0 too
        assert np.all(got.astype(np.float64) <= mn)
        inexact += int((got.astype(np.float64) < mn).sum())
    assert inexact > 0          # the case really exercises the rounding
    # scale and codes are computed from the STORED zero point, not from the exact minimum (the two
    # differ by up to one fp16 subnormal step here, a good part of a scale step)
    qmax = (1 << bits) - 1
    for vals, codes, scale, zero in ((kg, unpack(pk.k_codes, bits, g), pk.k_scale, pk.k_zero),
                                     (vg, unpack(pk.v_codes, bits, g), pk.v_scale, pk.v_zero)):
        zf, sf = f16_val(zero), f16_val(scale)
        quot = (vals.max(-1) - zf) / qmax
        gap = np.abs(quot - _f16_ceil(quot).astype(np.float64))
        clear = (gap == 0) | (gap > 4e-7 * quot)
        assert np.array_equal(scale.view(np.float16)[clear], _f16_ceil(quot)[clear])
        live = sf > 0
        ratio = (vals - zf[..., None])[live] / sf[live][:, None]
        want = np.clip(np.rint(ratio), 0, qmax)
        off_tie = np.abs(ratio - np.floor(ratio) - 0.5) > 1e-4
        assert np.array_equal(codes[live][off_tie], want[off_tie].astype(np.uint32))


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_codes_round_half_to_even(bits):
    # a group holding 0 and 2^B - 1 has zero 0 and scale 1 exactly; its other elements are the
    # half-integers 0.5, 1.5, 2.5, ... (bf16-exact below 128), whose quotients are exact ties
    g, D, L = 32, 32, 32
    qmax = (1 << bits) - 1
    halves = (np.arange(g - 2) % qmax) + 0.5                 # 0.5 .. qmax - 0.5, cyclic
    if bits == 8:
        halves = (np.arange(g - 2) * 4 % 127) + 0.5          # stay below 128 where x.5 is bf16-exact
    elems = np.concatenate([[0.0, float(qmax)], halves])
    assert np.array_equal(bf16_val(bf16_bits(elems)), elems)
    k = np.broadcast_to(elems[:, None], (1, 1, L, D)).copy()       # key groups run along tokens
    v = np.broadcast_to(elems[None, :], (1, 1, L, D)).copy()       # value groups run along channels
    pk, _, _, _ = _quant(k, v, bits, g)
    assert np.all(f16_val(pk.k_scale) == 1.0) and np.all(f16_val(pk.k_zero) == 0.0)
    want = np.concatenate([[0, qmax], 2 * np.floor((halves + 0.5) / 2)]).astype(np.uint32)   # nearest even
    assert np.any(want[2:] != np.floor(halves) + 1)          # differs from ties-away somewhere
    kc = unpack(pk.k_codes, bits, g)                         # [1,1,1,D,g]
    vc = unpack(pk.v_codes, bits, g)                         # [1,1,L,1,g]
    assert np.array_equal(kc[0, 0, 0], np.broadcast_to(want, (D, g)))
    assert np.array_equal(vc[0, 0, :, 0], np.broadcast_to(want, (L, g)))


def test_quantizer_dequant_formula_against_independent_unpack():
    bits, g, D = 4, 32, 64
    k = RNG.standard_normal((1, 1, 64, D)); v = RNG.standard_normal((1, 1, 64, D))
    pk, _, _, _ = _quant(k, v, bits, g)
    kd, vd = orc.dequantize(pk, D)
    kc = unpack(pk.k_codes, bits, g).astype(np.float64)          # [1,1,u,D,g]
    kref = kc * f16_val(pk.k_scale)[..., None] + f16_val(pk.k_zero)[..., None]
    kref = kref.transpose(0, 1, 2, 4, 3).reshape(1, 1, 64, D)    # (u, e) -> token
    vc = unpack(pk.v_codes, bits, g).astype(np.float64)          # [1,1,t,D/g,g]
    vref = (vc * f16_val(pk.v_scale)[..., None] + f16_val(pk.v_zero)[..., None]).reshape(1, 1, 64, D)
    assert np.array_equal(kd, kref) and np.array_equal(vd, vref)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_quantizer_lossless_cases(bits):
    g, D, L = 32, 32, 32
    qmax = (1 << bits) - 1
    kin = RNG.integers(0, qmax + 1, size=(1, 1, L, D)).astype(np.float64)
    vin = RNG.integers(0, qmax + 1, size=(1, 1, L, D)).astype(np.float64)
    kin[0, 0, 0, :] = 0; kin[0, 0, 1, :] = qmax       # K groups run along tokens
    vin[0, 0, :, 0] = 0; vin[0, 0, :, 1] = qmax       # V groups run along channels
    pk, kb, vb, _ = _quant(kin, vin, bits, g)
    kd, vd = orc.dequantize(pk, D)
    assert np.array_equal(kd, kin) and np.array_equal(vd, vin)
    assert np.all(f16_val(pk.k_scale) == 1.0) and np.all(f16_val(pk.k_zero) == 0.0)
    assert np.all(f16_val(pk.v_scale) == 1.0) and np.all(f16_val(pk.v_zero) == 0.0)
    # constant groups: scale 0, codes 0, exact reconstruction
    const = np.full((1, 1, L, D), 1.25)
    pk, _, _, _ = _quant(const, const, bits, g)
    kd, vd = orc.dequantize(pk, D)
    assert np.all(pk.k_codes == 0) and np.all(pk.k_scale == 0)
    assert np.array_equal(kd, const) and np.array_equal(vd, const)


def test_quantizer_axes_keys_per_channel_values_per_token():
    bits, g, D, L = 2, 32, 64, 64
    chan = RNG.standard_normal(D)
    tok = RNG.standard_normal(L)
    k = np.broadcast_to(chan[None, :], (1, 1, L, D)).copy()   # constant along tokens: lossless per-channel
    v = np.broadcast_to(tok[:, None], (1, 1, L, D)).copy()    # constant along channels: lossless per-token
    pk, kb, vb, _ = _quant(k, v, bits, g)
    kd, vd = orc.dequantize(pk, D)
    assert np.array_equal(kd, bf16_val(kb)) and np.array_equal(vd, bf16_val(vb))
    # swapped roles are lossy at 2 bits
    pk2, kb2, vb2, _ = _quant(v, k, bits, g)
    kd2, vd2 = orc.dequantize(pk2, D)
    assert not np.array_equal(kd2, bf16_val(kb2)) and not np.array_equal(vd2, bf16_val(vb2))


def test_quantizer_power_of_two_scaling_invariance():
    bits, g, D, L = 4, 32, 32, 64
    k = RNG.standard_normal((1, 1, L, D)); v = RNG.standard_normal((1, 1, L, D))
    pk1, _, _, _ = _quant(k, v, bits, g)
    pk2, _, _, _ = _quant(bf16_val(bf16_bits(k)) * 4.0, bf16_val(bf16_bits(v)) * 0.5, bits, g)
    assert np.array_equal(pk1.k_codes, pk2.k_codes) and np.array_equal(pk1.v_codes, pk2.v_codes)
    assert np.array_equal(f16_val(pk1.k_scale) * 4.0, f16_val(pk2.k_scale))
    assert np.array_equal(f16_val(pk1.v_zero) * 0.5, f16_val(pk2.v_zero))


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_pack_bit_positions(bits):
    g, D, L = 32, 32, 32
    qmax = (1 << bits) - 1
    per = 32 // bits
    for e in (0, 1, per - 1, per, g - 1):
        # K: token e of the group is the only maximum in channel 0 -> its code is qmax, others 0
        k = np.zeros((1, 1, L, D)); k[0, 0, e, 0] = 1.0
        v = np.zeros((1, 1, L, D)); v[0, 0, 0, e] = 1.0
        pk, _, _, _ = _quant(k, v, bits, g)
        exp_words = np.zeros(g * bits // 32, np.uint32)
        exp_words[e // per] = qmax << ((e % per) * bits)
        assert np.array_equal(pk.k_codes[0, 0, 0, 0], exp_words)
        assert np.array_equal(pk.v_codes[0, 0, 0, 0], exp_words)
        assert not pk.k_codes[0, 0, 0, 1:].any() and not pk.v_codes[0, 0, 1:].any()


def test_error_monotone_in_bits_and_gather_order():
    D, L, g = 64, 256, 32
    k = RNG.standard_normal((1, 1, L, D)); v = RNG.standard_normal((1, 1, L, D))
    kept = np.sort(RNG.choice(L, 64, replace=False)).astype(np.int32)[None, None]
    errs = []
    for bits in (2, 4, 8, 16):
        pk, kb, vb, _ = _quant(k, v, bits, g, kept)
        kd, vd = orc.dequantize(pk, D)
        ref = bf16_val(kb)[0, 0, kept[0, 0]]
        errs.append(np.abs(kd[0, 0] - ref).max())
    assert errs[0] > errs[1] > errs[2] > errs[3] == 0.0     # 16-bit is a pure gather


# ----------------------------------------------------------------------------- decode

def _dense_attention(q, K, V, G):
    Bt, Hq, D = q.shape
    out = np.zeros((Bt, Hq, D))
    for b in range(Bt):
        for h in range(Hq):
            a = K[b, h // G] @ q[b, h] / math.sqrt(D)
            p = np.exp(a - a.max()); p /= p.sum()
            out[b, h] = p @ V[b, h // G]
    return out


def test_decode_16bit_full_budget_equals_dense_attention():
    Bt, Hq, Hkv, D, L, w = 2, 8, 2, 64, 96, 8
    kb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    vb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    qwb = bf16_bits(RNG.standard_normal((Bt, Hq, w, D)))
    qb = bf16_bits(RNG.standard_normal((Bt, Hq, D)) * 2)
    pk, kept, _ = orc.compress_layer(kb, vb, qwb, budget_bits=16 * L, bits=16)
    assert pk.n == L and np.array_equal(kept[0, 0], np.arange(L))
    kd, vd = orc.dequantize(pk, D)
    out = orc.decode(qb, kd, vd)
    ref = _dense_attention(bf16_val(qb), bf16_val(kb), bf16_val(vb), Hq // Hkv)
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-14)


def test_decode_matches_dense_attention_on_dequantized_cache_and_q0_mean():
    Bt, Hq, Hkv, D, L, w = 1, 4, 2, 64, 256, 16
    kb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    vb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    qwb = bf16_bits(RNG.standard_normal((Bt, Hq, w, D)))
    qb = bf16_bits(RNG.standard_normal((Bt, Hq, D)))
    pk, kept, _ = orc.compress_layer(kb, vb, qwb, budget_bits=16 * 32, bits=4)
    assert pk.n == 128 and pk.n * 4 == 16 * 32
    kd, vd = orc.dequantize(pk, D)
    out = orc.decode(qb, kd, vd)
    assert np.allclose(out, _dense_attention(bf16_val(qb), kd, vd, Hq // Hkv), rtol=1e-12, atol=1e-14)
    out0 = orc.decode(np.zeros_like(qb), kd, vd)
    assert np.allclose(out0, vd.mean(2).repeat(Hq // Hkv, 1), rtol=1e-12, atol=1e-14)
    # order of the kept tokens does not matter at 16 bit (softmax attention is permutation invariant)
    pk16, kept16, _ = orc.compress_layer(kb, vb, qwb, budget_bits=16 * 32, bits=16)
    kd16, vd16 = orc.dequantize(pk16, D)
    perm = RNG.permutation(pk16.n)
    assert np.allclose(orc.decode(qb, kd16, vd16), orc.decode(qb, kd16[:, :, perm], vd16[:, :, perm]),
                       rtol=1e-12, atol=1e-14)


def test_budget_invariant_of_stored_bits():
    Bt, Hq, Hkv, D, L, w = 1, 4, 2, 64, 512, 32
    kb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    vb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    qwb = bf16_bits(RNG.standard_normal((Bt, Hq, w, D)))
    budget = 16 * 64
    for bits in (16, 8, 4, 2):
        pk, kept, _ = orc.compress_layer(kb, vb, qwb, budget, bits)
        assert pk.n * bits == budget
        code_bits = pk.k_codes.nbytes * 8 + pk.v_codes.nbytes * 8
        assert code_bits == 2 * Bt * Hkv * D * budget                     # tokens x bits held constant
        if bits < 16:
            meta_bits = 8 * (pk.k_scale.nbytes + pk.k_zero.nbytes + pk.v_scale.nbytes + pk.v_zero.nbytes)
            assert meta_bits == 2 * Bt * Hkv * D * pk.n * 32 // 32        # 32/g bits per element, g = 32
