"""GPU parity of the head-level budget path (KV heads of a layer keep different numbers of tokens): budgets, kept
indices and packed bytes bit for bit against the oracle, decode outputs within the decode tolerance."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import qp_oracle as orc
from paper_2412_12706_b200 import qp, synth
from tests.util import assert_packed_equal, bits_u16, cache_to_packed, check_kept_against_oracle, decode_tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("Bt,Hkv,P,w,n_mean,unit", [(2, 4, 992, 32, 256, 32), (1, 8, 8160, 32, 2048, 32),
                                                    (3, 3, 500, 8, 64, 8), (1, 2, 70000, 32, 4096, 64),
                                                    (2, 5, 200, 16, 216, 1), (1, 8, 40000, 32, 1024, 128)])
def test_budgets_bit_exact_with_ties_and_skew(Bt, Hkv, P, w, n_mean, unit):
    rng = np.random.default_rng(P + Hkv)
    s = rng.random((Bt, Hkv, P)).astype(np.float32)
    s[0, 0] *= 4.0                                      # a head that outranks the others
    s[0, Hkv - 1] = np.round(s[0, Hkv - 1] * 8) / 8     # heavy ties, within and across heads
    if Hkv > 2:
        s[0, 1] = np.round(s[0, 1] * 8) / 8
        s[Bt - 1, 2] *= 1e-3                            # a head that gets (almost) nothing
    want = orc.head_budgets(s.astype(np.float64), P + w, w, n_mean, unit)
    got = qp.head_budgets(torch.from_numpy(s).to(DEV), P + w, w, n_mean, unit)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy(), want)


@pytest.mark.parametrize("bits,group,k_axis,G", [(4, 32, 1, 4), (4, 64, 1, 4), (2, 32, 1, 2), (4, 32, 0, 4), (8, 32, 0, 8),
                                                 (16, 32, 0, 4)])
def test_layer_with_head_budgets_end_to_end(bits, group, k_axis, G):
    D, Hkv, L, w, n_mean = 128, 4, 2048 + 32, 32, 512
    wl = dataclasses.replace(synth.TINY, head_dim=D, n_kv_heads=Hkv, n_q_heads=Hkv * G, L=L, w=w, batch=2,
                             seed=synth.BASE_SEED + 90 + bits)
    k, v = synth.make_kv(wl, 0)
    qw = synth.make_q_win(wl, 0)
    qw[:, :G] *= 3.0                                    # sharper attention in KV head 0: its scores concentrate
    hc = qp.compress_layer_heads(k.to(DEV), v.to(DEV), qw.to(DEV), n_mean, bits, group, wl.pool, k_axis)
    torch.cuda.synchronize()
    pooled = orc.scores(bits_u16(qw), bits_u16(k), wl.pool)
    want_n = orc.head_budgets(pooled, L, w, n_mean, group)
    # budgets: the GPU ranks its own fp32 scores; allow the oracle's counts to differ by a unit only where a
    # near tie at the threshold decides (compare exactly when run on the GPU's scores, as done above)
    got_n = np.array(hc.n_heads).reshape(2, Hkv)
    assert np.all(got_n % group == 0) and got_n.sum() <= 2 * Hkv * n_mean
    assert np.abs(got_n - want_n).max() <= group and len(set(got_n.ravel().tolist())) > 1
    u16 = bits_u16
    for i, (c, kept) in enumerate(zip(hc.caches, hc.kept)):
        b, h = divmod(i, Hkv)
        n = hc.n_heads[i]
        swaps = check_kept_against_oracle(kept.cpu().numpy(), pooled[b:b + 1, h:h + 1], L, w, n)
        assert swaps <= 2
        kh, vh = u16(k[b:b + 1, h:h + 1]), u16(v[b:b + 1, h:h + 1])
        kept_np = kept.cpu().numpy()
        if bits == 16:
            ref = orc.quantize(kh, vh, kept_np, 16, group)
        else:
            ref = orc.quantize_ex(kh, vh, kept_np, bits, group, k_axis=k_axis)
        got = cache_to_packed(c)
        if k_axis == 1 and bits < 16:
            got.k_codes = c.k_codes.cpu().numpy().view(np.uint32).reshape(ref.k_codes.shape)
            got.k_scale, got.k_zero = u16(c.k_scale).reshape(ref.k_scale.shape), u16(c.k_zero).reshape(ref.k_zero.shape)
        assert_packed_equal(got, ref)
    # decode over the ragged heads against the oracle on the GPU's own caches
    q = synth.make_q_dec(wl, 0, 0)
    out = qp.decode_attn_heads(q.to(DEV), hc)
    torch.cuda.synchronize()
    outn = out.float().cpu().numpy()
    for i, (c, kept) in enumerate(zip(hc.caches, hc.kept)):
        b, h = divmod(i, Hkv)
        kh, vh = u16(k[b:b + 1, h:h + 1]), u16(v[b:b + 1, h:h + 1])
        ref = orc.quantize(kh, vh, kept.cpu().numpy(), 16, group) if bits == 16 else \
            orc.quantize_ex(kh, vh, kept.cpu().numpy(), bits, group, k_axis=k_axis)
        kd, vd = orc.dequantize(ref, D)
        want = orc.decode(u16(q[b:b + 1, h * G:(h + 1) * G]), kd, vd)
        err = float(np.abs(outn[b, h * G:(h + 1) * G] - want[0]).max())
        assert err <= decode_tolerance(want), (i, err)
