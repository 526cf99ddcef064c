"""GPU parity of the other quantization strategies (Sec. 5.3 "Quantization methods"): keys grouped per token
(the FlexGen arrangement) and outlier filtering with 16-bit side lists, through the C ABI against the CPU oracle.
Packed bytes and side lists must match bit for bit, decode outputs within the decode tolerance."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import qp_oracle as orc
from paper_2412_12706_b200 import qp, synth
from tests.util import assert_packed_equal, bits_u16, cache_to_packed, decode_tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(D, G, L, batch=2, Hkv=2, seed_off=0):
    wl = dataclasses.replace(synth.TINY, head_dim=D, n_kv_heads=Hkv, n_q_heads=Hkv * G, L=L, batch=batch,
                             seed=synth.BASE_SEED + 70 + seed_off)
    k, v = synth.make_kv(wl, 0)                         # 4 key channels x10: plenty of |x| > 6
    v[0, 0, 5, 3] = 31.0                                # a few value outliers too
    v[batch - 1, Hkv - 1, ::9, D - 1] = -7.5
    return wl, k, v


def _side_np(bufs):
    idx, val, cnt, tp = bufs
    return idx.cpu().numpy(), bits_u16(val), cnt.cpu().numpy(), tp.cpu().numpy()


@pytest.mark.parametrize("bits,group,D,G,k_axis,thr", [
    (4, 32, 128, 4, 1, None), (4, 64, 128, 4, 1, None), (2, 32, 128, 4, 1, None), (8, 32, 64, 2, 1, None),
    (4, 32, 64, 8, 1, None), (4, 128, 128, 2, 1, None), (4, 64, 64, 3, 1, None), (4, 32, 128, 8, 1, None),
    (4, 32, 128, 4, 0, 6.0), (4, 64, 128, 4, 1, 6.0), (2, 32, 64, 8, 1, 6.0), (8, 128, 128, 1, 0, 6.0),
    (2, 32, 128, 3, 0, 6.0)])
def test_quantize_and_decode_under_a_strategy(bits, group, D, G, k_axis, thr):
    n, L = 384, 1000
    wl, k, v = _inputs(D, G, L, seed_off=bits + group + k_axis)
    rng = np.random.default_rng(bits * 100 + group)
    kept = np.stack([np.sort(rng.choice(L, n, replace=False)) for _ in range(wl.batch * wl.n_kv_heads)])
    kept = kept.reshape(wl.batch, wl.n_kv_heads, n).astype(np.int32)
    ref = orc.quantize_ex(bits_u16(k), bits_u16(v), kept, bits, group, k_axis=k_axis, outlier_threshold=thr)

    cache = qp.alloc_cache(wl.batch, wl.n_q_heads, wl.n_kv_heads, D, bits, group, n, DEV)
    if k_axis == 1:                                     # key arrays take the value arrays' shapes (same sizes)
        cache.k_codes = cache.k_codes.view(wl.batch, wl.n_kv_heads, n, D // group, group * bits // 32)
        cache.k_scale = cache.k_scale.view(wl.batch, wl.n_kv_heads, n, D // group)
        cache.k_zero = cache.k_zero.view(wl.batch, wl.n_kv_heads, n, D // group)
    st = qp.make_strategy(cache, k_axis, thr)
    qp.gather_quantize_ex(k.to(DEV), v.to(DEV), torch.from_numpy(kept).to(DEV), cache, st)
    torch.cuda.synchronize()
    got = cache_to_packed(cache)
    if k_axis == 1:                                     # (the helper slices key arrays by token groups)
        got.k_codes = cache.k_codes.cpu().numpy().view(np.uint32).reshape(ref.k_codes.shape)
        got.k_scale, got.k_zero = bits_u16(cache.k_scale), bits_u16(cache.k_zero)
    assert_packed_equal(got, ref)
    if thr is not None:
        for bufs, side in zip(st.bufs, (ref.k_side, ref.v_side)):
            idx, val, cnt, tp = _side_np(bufs)
            assert np.array_equal(cnt, side.cnt) and cnt.min() >= 0
            for b in range(wl.batch):
                for h in range(wl.n_kv_heads):
                    c = int(cnt[b, h])
                    assert np.array_equal(idx[b, h, :c], side.idx[b, h, :c])
                    assert np.array_equal(val[b, h, :c], side.val[b, h, :c])
                    want_tp = np.searchsorted(side.idx[b, h, :c], 32 * D * np.arange(n // 32 + 1))
                    assert np.array_equal(tp[b, h], want_tp.astype(np.int32))
        assert ref.k_side.cnt.sum() > 100 and ref.v_side.cnt.sum() > 0

    kd, vd = orc.dequantize(ref, D)
    for step in range(2):
        q = synth.make_q_dec(wl, 0, step)
        out = qp.decode_attn_ex(q.to(DEV), cache, st)
        torch.cuda.synchronize()
        want = orc.decode(bits_u16(q), kd, vd)
        err = float(np.abs(out.float().cpu().numpy() - want).max())
        assert err <= decode_tolerance(want), (step, err)
        # the chunked kernel dequantizes in fp32: far inside the stated tolerance, and close enough that a
        # dropped or misplaced outlier (|delta| > 6 on a logit or a value) would show
        assert err <= 2e-2 * max(1.0, float(np.abs(want).max())), (step, err)


def test_strategy_without_filtering_on_the_channel_axis_matches_the_plain_calls():
    wl, k, v = _inputs(128, 4, 700)
    n, bits, group = 256, 4, 32
    kept = torch.arange(n, dtype=torch.int32).expand(wl.batch, wl.n_kv_heads, n).contiguous().to(DEV)
    a = qp.alloc_cache(wl.batch, wl.n_q_heads, wl.n_kv_heads, 128, bits, group, n, DEV)
    b = qp.alloc_cache(wl.batch, wl.n_q_heads, wl.n_kv_heads, 128, bits, group, n, DEV)
    qp.gather_quantize(k.to(DEV), v.to(DEV), kept, a)
    st = qp.make_strategy(b, 0, None)
    qp.gather_quantize_ex(k.to(DEV), v.to(DEV), kept, b, st)
    torch.cuda.synchronize()
    assert_packed_equal(cache_to_packed(a), cache_to_packed(b))
    q = synth.make_q_dec(wl, 0, 0).to(DEV)
    x, y = qp.decode_attn(q, a), qp.decode_attn_ex(q, b, st)
    torch.cuda.synchronize()
    assert float((x.float() - y.float()).abs().max()) <= 2e-2


def test_side_list_overflow_is_reported_not_written_past_the_end():
    wl, k, v = _inputs(64, 2, 300, batch=1, Hkv=1)
    n = 128
    kept = torch.arange(n, dtype=torch.int32).expand(1, 1, n).contiguous().to(DEV)
    cache = qp.alloc_cache(1, 2, 1, 64, 4, 32, n, DEV)
    st = qp.make_strategy(cache, 0, 6.0, cap=8)                      # far too small for the outlier channels
    # the lists are views of larger buffers whose remainder must stay untouched
    big = [torch.full((64,), -7, dtype=torch.int32, device=DEV), torch.full((64,), -7.0, dtype=torch.bfloat16, device=DEV)]
    st.desc.k_side.idx, st.desc.k_side.val = big[0].data_ptr(), big[1].data_ptr()
    qp.gather_quantize_ex(k.to(DEV), v.to(DEV), kept, cache, st)
    torch.cuda.synchronize()
    assert int(st.bufs[0][2][0, 0]) == -1                            # keys: overflow flagged
    assert bool((big[0][8:] == -7).all()) and bool((big[1][8:] == -7.0).all()) and bool((big[0][:8] >= 0).all())


def test_strategy_arguments_are_checked_before_any_launch():
    c = qp.cache_layout(1, 4, 1, 128, 16, 32, 64)
    fake = 0x10000
    c.k_codes = c.v_codes = fake
    s = qp.qp_strategy()
    import ctypes
    assert qp.lib().qp_decode_attn_ex(fake, ctypes.byref(c), ctypes.byref(s), fake, fake, 1 << 20, None) == 2   # 16 bit
    c4 = qp.cache_layout(1, 4, 1, 128, 4, 32, 64)
    c4.k_codes = c4.v_codes = c4.k_scale = c4.k_zero = c4.v_scale = c4.v_zero = fake
    s.k_axis = 2
    assert qp.lib().qp_decode_attn_ex(fake, ctypes.byref(c4), ctypes.byref(s), fake, fake, 1 << 20, None) == 1
    s.k_axis, s.outlier_threshold = 1, 6.0                            # filtering on, side lists missing
    assert qp.lib().qp_gather_quantize_ex(fake, fake, fake, 100, ctypes.byref(c4), ctypes.byref(s), None) == 1
    torch.cuda.synchronize()
