"""Pins of the oracle's other quantization strategies (Sec. 5.3 "Quantization methods"; Appendix B
"KV quantization"): keys grouped token by token like the values (the FlexGen arrangement) and outlier
filtering (numbers whose absolute value exceeds a threshold are excluded from quantization and kept
in 16 bit).  Expected values come from numpy, from closed forms or from the already pinned KIVI path,
never from the functions under test.
"""
import math

import numpy as np
import pytest

from oracle import qp_oracle as orc
from tests.test_oracle_pins import RNG, bf16_bits, bf16_val, f16_val, unpack, _f16_ceil, _f16_floor


def _ident(Bt, Hkv, n):
    return np.broadcast_to(np.arange(n, dtype=np.int32), (Bt, Hkv, n)).copy()


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_no_filtering_and_channel_axis_is_the_kivi_quantizer_bit_for_bit(bits):
    Bt, Hkv, L, D, g = 2, 2, 96, 64, 32
    kb, vb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)) * 3), bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    kept = np.sort(RNG.choice(L, 64, replace=False)).astype(np.int32)[None, None].repeat(Bt, 0).repeat(Hkv, 1)
    a = orc.quantize(kb, vb, kept, bits, g)
    b = orc.quantize_ex(kb, vb, kept, bits, g, k_axis=0, outlier_threshold=None)
    for f in ("k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero"):
        assert np.array_equal(getattr(a, f), getattr(b, f)), f
    c = orc.quantize_ex(kb, vb, kept, bits, g, k_axis=0, outlier_threshold=1e30)     # nothing exceeds it
    assert np.array_equal(a.k_codes, c.k_codes) and np.array_equal(a.v_scale, c.v_scale)
    assert not c.k_side.cnt.any() and not c.v_side.cnt.any()


@pytest.mark.parametrize("bits,g", [(4, 32), (2, 64), (8, 32)])
def test_token_axis_keys_are_quantized_exactly_like_values(bits, g):
    """Keys grouped per token = the value rule applied to the key tensor: feed K in as V of the pinned path."""
    Bt, Hkv, L, D = 1, 2, 64, 128
    kb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)) * 2)
    vb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    kept = _ident(Bt, Hkv, L)
    tok = orc.quantize_ex(kb, vb, kept, bits, g, k_axis=1)
    via_values = orc.quantize(vb, kb, kept, bits, g)                 # roles swapped: K travels as "V"
    assert tok.k_codes.shape == (Bt, Hkv, L, D // g, g * bits // 32)
    assert np.array_equal(tok.k_codes, via_values.v_codes)
    assert np.array_equal(tok.k_scale, via_values.v_scale) and np.array_equal(tok.k_zero, via_values.v_zero)
    kd, vd = orc.dequantize(tok, D)
    kd2, _ = orc.dequantize(via_values, D)                           # its "V" output is our K
    assert np.array_equal(kd, _)
    # axis pin: keys constant along the channels of a token are lossless token by token, lossy per channel
    row = RNG.standard_normal(L)
    kconst = bf16_bits(np.broadcast_to(row[:, None], (1, 1, L, D)))
    t = orc.quantize_ex(kconst, vb[:, :1], kept[:, :1], 2, 32, k_axis=1)
    assert np.array_equal(orc.dequantize(t, D)[0], bf16_val(kconst))
    c = orc.quantize_ex(kconst, vb[:, :1], kept[:, :1], 2, 32, k_axis=0)
    assert not np.array_equal(orc.dequantize(c, D)[0], bf16_val(kconst))


@pytest.mark.parametrize("k_axis", [0, 1])
@pytest.mark.parametrize("bits", [2, 4])
def test_outliers_are_listed_in_order_kept_exactly_and_left_out_of_the_range(bits, k_axis):
    Bt, Hkv, L, D, g, thr = 2, 2, 64, 64, 32, 6.0
    k = RNG.standard_normal((Bt, Hkv, L, D)); k[..., 5] *= 8; k[..., 40] *= 8       # two outlier channels
    v = RNG.standard_normal((Bt, Hkv, L, D)); v[0, 1, 7, 3] = -50.0; v[1, 0, 63, 63] = 6.0   # 6.0 itself is NOT one
    kb, vb = bf16_bits(k), bf16_bits(v)
    kept = _ident(Bt, Hkv, L)
    pk = orc.quantize_ex(kb, vb, kept, bits, g, k_axis=k_axis, outlier_threshold=thr)
    kd, vd = orc.dequantize(pk, D)
    qmax = (1 << bits) - 1
    for name, xb, side, xd, scale, zero, axis in (("k", kb, pk.k_side, kd, pk.k_scale, pk.k_zero, k_axis),
                                                  ("v", vb, pk.v_side, vd, pk.v_scale, pk.v_zero, 1)):
        x = bf16_val(xb)
        out = np.abs(x) > thr
        for b in range(Bt):
            for h in range(Hkv):
                want = np.flatnonzero(out[b, h].ravel())                           # ascending t*D + d
                c = int(side.cnt[b, h])
                assert c == len(want)
                assert np.array_equal(side.idx[b, h, :c], want.astype(np.int32))
                assert np.array_equal(side.val[b, h, :c], xb[b, h].ravel()[want])
        assert np.array_equal(xd[out], x[out])                                     # exact reconstruction
        # groups: [.., n_groups, g] views of values / masks, per token or per channel
        if axis == 1:
            view = lambda a: a.reshape(Bt, Hkv, L, D // g, g)
        else:
            view = lambda a: a.reshape(Bt, Hkv, L // g, g, D).transpose(0, 1, 2, 4, 3)
        xg, og, dg = view(x), view(out), view(xd)
        zf, sf = f16_val(zero), f16_val(scale)
        inl_min = np.where(og, np.inf, xg).min(-1)
        inl_max = np.where(og, -np.inf, xg).max(-1)
        some = np.isfinite(inl_min)
        assert np.array_equal(zero.view(np.float16)[some], _f16_floor(inl_min[some]))   # range from inliers only
        quot = (inl_max[some] - zf[some]) / qmax
        gap = np.abs(quot - _f16_ceil(quot).astype(np.float64))
        clear = (gap == 0) | (gap > 4e-7 * quot)
        assert np.array_equal(scale.view(np.float16)[some][clear], _f16_ceil(quot)[clear])
        assert np.all(sf[~some] == 0) and np.all(zf[~some] == 0)                   # a group of outliers only
        err = np.abs(dg - xg)
        assert np.all(err[~og] <= (sf[..., None] / 2 * (1 + 1e-3)).repeat(g, -1)[~og])
    assert pk.v_side.cnt.sum() == 1                                                # only the -50


def test_filtering_shrinks_the_scale_of_a_group_with_one_large_element():
    """Closed form: 31 values in {0, 1/4, .., 1} plus one 100.  With filtering the group's range is [0, 1]
    (scale 1/15 rounded up to fp16 at 4 bit), without it [0, 100]."""
    D, L, g, bits = 32, 32, 32, 4
    row = (np.arange(g) % 5) / 4.0
    row[0], row[1], row[17] = 0.0, 1.0, 100.0
    v = np.broadcast_to(row[None, :], (1, 1, L, D)).copy()
    k = np.broadcast_to(row[:, None], (1, 1, L, D)).copy()                         # key groups run along tokens
    kept = _ident(1, 1, L)
    f = orc.quantize_ex(bf16_bits(k), bf16_bits(v), kept, bits, g, k_axis=0, outlier_threshold=6.0)
    u = orc.quantize_ex(bf16_bits(k), bf16_bits(v), kept, bits, g, k_axis=0, outlier_threshold=None)
    want_f = float(_f16_ceil(np.array([1.0 / 15]))[0]); want_u = float(_f16_ceil(np.array([100.0 / 15]))[0])
    assert np.all(f16_val(f.v_scale) == want_f) and np.all(f16_val(f.k_scale) == want_f)
    assert np.all(f16_val(u.v_scale) == want_u) and np.all(f16_val(u.k_scale) == want_u)
    assert f.v_side.cnt[0, 0] == L and f.k_side.cnt[0, 0] == D                     # one per value row / key channel
    kd, vd = orc.dequantize(f, D)
    assert vd[0, 0, 3, 17] == 100.0 and kd[0, 0, 17, 9] == 100.0
    assert abs(vd[0, 0, 3, 2] - row[2]) <= want_f / 2 * 1.001


def test_decode_over_a_filtered_cache_is_dense_attention_over_its_reconstruction():
    Bt, Hq, Hkv, D, L = 1, 4, 2, 64, 96
    k = RNG.standard_normal((Bt, Hkv, L, D)); k[..., 11] *= 9
    v = RNG.standard_normal((Bt, Hkv, L, D)); v[0, 0, ::7, 2] = 12.0
    qb = bf16_bits(RNG.standard_normal((Bt, Hq, D)))
    pk = orc.quantize_ex(bf16_bits(k), bf16_bits(v), _ident(Bt, Hkv, L), 4, 32, k_axis=1, outlier_threshold=6.0)
    kd, vd = orc.dequantize(pk, D)
    out = orc.decode(qb, kd, vd)
    q = bf16_val(qb)
    for h in range(Hq):
        a = kd[0, h // 2] @ q[0, h] / math.sqrt(D)
        p = np.exp(a - a.max()); p /= p.sum()
        assert np.allclose(out[0, h], p @ vd[0, h // 2], rtol=1e-12, atol=1e-14)
    # the outlier channel is exact, so the filtered cache is closer to the bf16 keys than the unfiltered one
    un = orc.quantize_ex(bf16_bits(k), bf16_bits(v), _ident(Bt, Hkv, L), 4, 32, k_axis=1)
    kd_un, _ = orc.dequantize(un, D)
    kx = bf16_val(bf16_bits(k))
    assert np.abs(kd - kx).max() < 0.5 * np.abs(kd_un - kx).max()
