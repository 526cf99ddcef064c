"""Pins of the oracle's decode-time append (Eq. 2 on a quantized-pruned cache).

Expected values come from numpy dense attention over explicitly built key/value matrices, from
exactly representable (lossless) groups and from counting; none comes from the append oracle
itself or from the CUDA path.
"""
import math

import numpy as np
import pytest
import torch

from oracle import qp_oracle as orc

RNG = np.random.default_rng(2412127)


def bf16_bits(x):
    t = torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_val(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def dense_attention(q, K, V, G):
    Bt, Hq, D = q.shape
    out = np.zeros((Bt, Hq, D))
    for b in range(Bt):
        for h in range(Hq):
            a = K[b, h // G] @ q[b, h] / math.sqrt(D)
            p = np.exp(a - a.max()); p /= p.sum()
            out[b, h] = p @ V[b, h // G]
    return out


def prompt_cache(bits, g, Bt=1, Hq=4, Hkv=2, D=64, L=192, w=16, n16=None):
    kb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    vb = bf16_bits(RNG.standard_normal((Bt, Hkv, L, D)))
    qwb = bf16_bits(RNG.standard_normal((Bt, Hq, w, D)))
    budget = bits * (n16 if n16 is not None else 2 * max(g, 32))
    pk, kept, _ = orc.compress_layer(kb, vb, qwb, budget, bits, g)
    return kb, vb, pk, kept


def test_16bit_appends_equal_dense_attention_over_the_concatenation():
    Bt, Hq, Hkv, D = 2, 8, 2, 64
    kb, vb, pk, kept = prompt_cache(16, 32, Bt, Hq, Hkv, D, L=96, w=8, n16=40)
    st = orc.gen_state(pk, D)
    K = np.stack([[bf16_val(kb)[b, h, kept[b, h]] for h in range(Hkv)] for b in range(Bt)])
    V = np.stack([[bf16_val(vb)[b, h, kept[b, h]] for h in range(Hkv)] for b in range(Bt)])
    for step in range(5):
        kn = bf16_bits(RNG.standard_normal((Bt, Hkv, D)))
        vn = bf16_bits(RNG.standard_normal((Bt, Hkv, D)))
        st = orc.append(st, kn, vn)
        K = np.concatenate([K, bf16_val(kn)[:, :, None]], axis=2)
        V = np.concatenate([V, bf16_val(vn)[:, :, None]], axis=2)
        assert st.n_tail == 0 and st.packed.n == 40 + step + 1        # 16 bit: nothing waits in a tail
        qb = bf16_bits(RNG.standard_normal((Bt, Hq, D)) * 2)
        assert np.allclose(orc.decode_state(qb, st, D), dense_attention(bf16_val(qb), K, V, Hq // Hkv),
                           rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("bits,g", [(4, 32), (2, 32), (8, 64), (4, 64)])
def test_tail_is_exact_and_lossless_groups_flush_exactly(bits, g):
    """Tokens with integer entries in [0, 2^B - 1] whose every group holds both 0 and 2^B - 1
    quantize without loss (scale 1, zero 0), so before AND after the flush the result must be dense
    attention over [dequantized prompt cache ; the appended rows themselves]."""
    Bt, Hq, Hkv, D = 1, 4, 2, 64
    qmax = (1 << bits) - 1
    kb, vb, pk, kept = prompt_cache(bits, g, Bt, Hq, Hkv, D)
    K, V = orc.dequantize(pk, D)
    n0 = pk.n
    st = orc.gen_state(pk, D)
    new_k = RNG.integers(0, qmax + 1, (g + 5, Bt, Hkv, D)).astype(np.float64)
    new_v = RNG.integers(0, qmax + 1, (g + 5, Bt, Hkv, D)).astype(np.float64)
    new_k[3] = 0; new_k[7] = qmax                   # every key group (a channel over g tokens) spans 0..qmax
    new_v[..., 0::g] = 0; new_v[..., 1::g] = qmax   # every value group (g channels of a token) too
    for t in range(g + 5):
        st = orc.append(st, bf16_bits(new_k[t]), bf16_bits(new_v[t]))
        K = np.concatenate([K, new_k[t][:, :, None]], axis=2)
        V = np.concatenate([V, new_v[t][:, :, None]], axis=2)
        assert st.n_tail == (t + 1) % g
        assert st.packed.n == n0 + g * ((t + 1) // g)
        if t in (0, g - 2, g - 1, g, g + 4):
            qb = bf16_bits(RNG.standard_normal((Bt, Hq, D)) * 0.3)
            assert np.allclose(orc.decode_state(qb, st, D), dense_attention(bf16_val(qb), K, V, Hq // Hkv),
                               rtol=1e-12, atol=1e-14)
    # the flushed group's stored parameters are the lossless ones
    u = n0 // g
    assert np.all(st.packed.k_scale[:, :, u].view(np.float16) == 1.0)
    assert np.all(st.packed.k_zero[:, :, u].view(np.float16) == 0.0)
    assert np.all(st.packed.v_scale[:, :, n0:n0 + g].view(np.float16) == 1.0)


def test_zero_query_gives_the_mean_over_packed_and_tail_tokens():
    bits, g, D = 4, 32, 64
    kb, vb, pk, kept = prompt_cache(bits, g, D=D)
    st = orc.gen_state(pk, D)
    vs = []
    for t in range(7):
        vn = bf16_bits(RNG.standard_normal((1, 2, D)))
        st = orc.append(st, bf16_bits(RNG.standard_normal((1, 2, D))), vn)
        vs.append(bf16_val(vn))
    _, vd = orc.dequantize(pk, D)
    allv = np.concatenate([vd, np.stack(vs, axis=2)], axis=2)            # [1,2,n+7,D]
    out = orc.decode_state(np.zeros((1, 4, D), np.uint16), st, D)
    assert np.allclose(out, allv.mean(2).repeat(2, 1), rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("bits,g", [(4, 32), (2, 32), (8, 128)])
def test_flushed_group_equals_the_prompt_quantizer_on_the_same_tokens(bits, g):
    """Appending g tokens must leave the cache that S3 builds when those g tokens are the last kept
    tokens of a longer prompt: same codes, scales and zeros, group for group."""
    Bt, Hkv, D, L = 1, 2, 128, 256
    kb = bf16_bits(RNG.standard_normal((Bt, Hkv, L + g, D)) * 3)
    vb = bf16_bits(RNG.standard_normal((Bt, Hkv, L + g, D)))
    kept = np.sort(RNG.choice(L, 2 * g, replace=False)).astype(np.int32)
    kept = np.broadcast_to(kept, (Bt, Hkv, 2 * g)).copy()
    st = orc.gen_state(orc.quantize(kb[:, :, :L], vb[:, :, :L], kept, bits, g), D)
    for t in range(g):
        st = orc.append(st, kb[:, :, L + t], vb[:, :, L + t])
    kept_all = np.concatenate([kept, np.broadcast_to(np.arange(L, L + g, dtype=np.int32), (Bt, Hkv, g))], axis=2)
    ref = orc.quantize(kb, vb, kept_all, bits, g)
    assert st.n_tail == 0 and st.packed.n == ref.n
    for name in ("k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero"):
        assert np.array_equal(getattr(st.packed, name), getattr(ref, name)), name
