"""Parity at the full sizes of the benchmark configurations, in the launch configuration the
benchmark times (qp_compress_layer per layer, qp_decode_attn_layers over the layers).

The oracle cannot redo a whole 32k x 8-batch layer in seconds, so the GPU runs the full problem
and the oracle recomputes SAMPLED (batch, KV head) pairs from the same inputs: indices with the
near-tie rule, packed bytes bit for bit on the GPU's indices, decode outputs within tolerance.
Everything not sampled is covered by structural properties that hold at any size."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import qp_oracle as orc
from paper_2412_12706_b200 import qp, synth
from tests.util import assert_packed_equal, bits_u16, check_kept_against_oracle, decode_tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _slice_packed(cache, b, hk):
    """Packed arrays of one (batch, KV head) pair as an oracle Packed with Bt = Hkv = 1."""
    d = cache.desc
    n, ng = d.n_keep, d.n_keep // d.group                       # tokens / key groups in use (the arrays may have room for more)
    sl = lambda t, m: t[b:b + 1, hk:hk + 1, :m].contiguous()
    if d.bits == 16:
        return orc.Packed(16, d.group, n, bits_u16(sl(cache.k_codes, n)), bits_u16(sl(cache.v_codes, n)),
                          None, None, None, None)
    u32 = lambda t, m: sl(t, m).cpu().numpy().view(np.uint32)
    return orc.Packed(d.bits, d.group, n, u32(cache.k_codes, ng), u32(cache.v_codes, n),
                      bits_u16(sl(cache.k_scale, ng)), bits_u16(sl(cache.k_zero, ng)),
                      bits_u16(sl(cache.v_scale, n)), bits_u16(sl(cache.v_zero, n)))


def _check_structure(kept: torch.Tensor, L: int, w: int):
    """Holds for every head at any size: ascending, unique, in range, window last."""
    k = kept.long()
    assert bool((k[..., 1:] > k[..., :-1]).all())
    assert int(k.min()) >= 0 and int(k.max()) == L - 1
    assert bool((k[..., -w:] == torch.arange(L - w, L, device=k.device)).all())


def run_fullsize(wl: synth.Workload, layers, samples, variants=None, decode_steps=2):
    """variants: list of (bits, tokens16) sharing the same K, V, Q_win (the constant-memory sweep)."""
    variants = variants or [(wl.bits, wl.tokens16)]
    G = wl.n_q_heads // wl.n_kv_heads
    per_variant = {v: {"caches": [], "kept": []} for v in variants}
    host = {}                                                   # sampled inputs per layer
    pooled_ref = {}
    for layer in layers:
        k, v = synth.make_kv(wl, layer, device=DEV)
        qw = synth.make_q_win(wl, layer, device=DEV)
        ws = torch.empty(qp.compress_workspace_bytes(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.L, wl.w),
                         dtype=torch.uint8, device=DEV)
        for bits, tokens16 in variants:
            wv = dataclasses.replace(wl, bits=bits, tokens16=tokens16)
            cache, kept = qp.compress_layer(k, v, qw, wv.layer_budget_bits(layer), bits, wl.group, wl.pool, workspace=ws)
            _check_structure(kept, wl.L, wl.w)
            assert kept.shape[-1] * bits <= wv.layer_budget_bits(layer)
            per_variant[(bits, tokens16)]["caches"].append(cache)
            per_variant[(bits, tokens16)]["kept"].append(kept)
        # pull the sampled pairs to the host as a pseudo batch [S,1,L,D] (the oracle threads over it)
        ks = torch.stack([k[b, hk] for b, hk in samples])[:, None].contiguous()
        vs = torch.stack([v[b, hk] for b, hk in samples])[:, None].contiguous()
        qs = torch.stack([qw[b, hk * G:(hk + 1) * G] for b, hk in samples]).contiguous()
        host[layer] = (bits_u16(ks), bits_u16(vs), bits_u16(qs))
        pooled_ref[layer] = orc.scores(host[layer][2], host[layer][0], wl.pool)
        del k, v, qw, ks, vs, qs
    torch.cuda.synchronize()

    swaps = 0
    for (bits, tokens16), pv in per_variant.items():
        # decode all layers in one launch pair, as the benchmark does
        qd = [[synth.make_q_dec(wl, layer, s, device=DEV) for layer in layers] for s in range(decode_steps)]
        outs = [[torch.empty_like(q) for q in row] for row in qd]
        for s in range(decode_steps):
            qp.decode_attn_layers(qp.LayerBatch(qd[s], pv["caches"], outs[s]))
        torch.cuda.synchronize()
        for li, layer in enumerate(layers):
            cache, kept = pv["caches"][li], pv["kept"][li]
            n = kept.shape[-1]
            kb, vb, qb = host[layer]
            kept_s = np.stack([kept[b, hk].cpu().numpy() for b, hk in samples])[:, None]
            swaps += check_kept_against_oracle(kept_s, pooled_ref[layer], wl.L, wl.w, n)
            ref = orc.quantize(kb, vb, kept_s, bits, wl.group)
            for si, (b, hk) in enumerate(samples):
                got = _slice_packed(cache, b, hk)
                one = orc.Packed(ref.bits, ref.group, ref.n, ref.k_codes[si:si + 1], ref.v_codes[si:si + 1],
                                 *(None if a is None else a[si:si + 1] for a in (ref.k_scale, ref.k_zero,
                                                                                 ref.v_scale, ref.v_zero)))
                assert_packed_equal(got, one)
            kd, vd = orc.dequantize(ref, wl.head_dim)
            for s in range(decode_steps):
                qh = torch.stack([qd[s][li][b, hk * G:(hk + 1) * G] for b, hk in samples])    # [S,G,D]
                ref_out = orc.decode(bits_u16(qh), kd, vd)
                got_out = torch.stack([outs[s][li][b, hk * G:(hk + 1) * G] for b, hk in samples]).float().cpu().numpy()
                assert np.abs(got_out - ref_out).max() <= decode_tolerance(ref_out)
                assert bool(torch.isfinite(outs[s][li].float()).all())
    return swaps


def test_llama8b_32k_batch8_2bit_rotary_full_layer():
    swaps = run_fullsize(synth.LLAMA8B_32K_B8, layers=[0, 31], samples=[(0, 0), (3, 5), (7, 7)])
    assert swaps <= 6


def test_llama8b_128k_constant_memory_sweep_full_layer():
    wl = synth.sweep_128k(4)
    variants = [(16, 1024), (8, 1024), (4, 1024), (2, 1024)]      # (B,16) (2B,8) (4B,4) (8B,2) with B = 1024
    swaps = run_fullsize(wl, layers=[5], samples=[(0, 2)], variants=variants)
    assert swaps <= 8


def test_llama70b_pyramid_first_and_last_layer():
    wl = synth.LLAMA70B_32K_B4
    assert wl.n_keep(0) == 8192 and wl.n_keep(79) == 2048          # 2x .. 0.5x of the 4096-token mean
    swaps = run_fullsize(wl, layers=[0, 79], samples=[(0, 0), (3, 6)])
    assert swaps <= 4


def test_llama70b_pyramid_with_the_papers_window_of_8():
    """The same 70B-shape pyramid layers with the observation window the paper uses for PyramidKV (the last 8
    tokens, Appendix B "KV eviction methods") instead of 32, at full size."""
    wl = dataclasses.replace(synth.LLAMA70B_32K_B4, w=8)
    swaps = run_fullsize(wl, layers=[0, 79], samples=[(1, 3), (2, 7)], decode_steps=1)
    assert swaps <= 4


def test_llama8b_generation_loop_in_the_bench_configuration():
    """Append + decode over packed tokens and tail at the benchmark's launch shape: 128 layer descriptors
    (32 layers of 4 sequences) per qp_append_kv_layers / qp_decode_attn_tail_layers call, tails cycling
    through a flush.  The oracle follows SAMPLED (descriptor, KV head) pairs from the GPU's own prompt caches;
    every output is checked for finiteness and every descriptor for its counters."""
    wl = synth.LLAMA8B_8K
    n_seq, nl, g, D, Hkv = 4, wl.n_layers, wl.group, wl.head_dim, wl.n_kv_heads
    G = wl.n_q_heads // Hkv
    steps = g + 3
    caches, tails = [], []
    ws = torch.empty(qp.compress_workspace_bytes(wl.batch, wl.n_q_heads, Hkv, D, wl.L, wl.w), dtype=torch.uint8, device=DEV)
    for s in range(n_seq):
        wls = dataclasses.replace(wl, seed=wl.seed + 1000 * s)
        for l in range(nl):
            k, v = synth.make_kv(wls, l, device=DEV)
            qw = synth.make_q_win(wls, l, device=DEV)
            c, _ = qp.compress_layer(k, v, qw, wl.budget_bits, wl.bits, g, wl.pool, workspace=ws, n_cap=wl.n_keep(l) + 2 * g)
            caches.append(c); tails.append(qp.alloc_tail(c))
    n_desc = len(caches)
    samples = [(0, 0), (37, 5), (n_desc - 1, 7)]                  # (descriptor, KV head)
    torch.cuda.synchronize()
    states = [orc.gen_state(_slice_packed(caches[i], 0, hk), D) for i, hk in samples]
    mk = lambda *shape: [torch.empty(shape, dtype=torch.bfloat16, device=DEV) for _ in range(n_desc)]
    kn, vn, qs, outs = mk(1, Hkv, D), mk(1, Hkv, D), mk(1, wl.n_q_heads, D), mk(1, wl.n_q_heads, D)
    gb = qp.GenBatch(qs, kn, vn, caches, tails, outs)
    for st in range(steps):
        # one stream of seeded rows per step, cut into the descriptors' tensors
        rows = synth.normal_f32(wl.seed + 77, 0, 100 + st, n_desc * (2 * Hkv + wl.n_q_heads) * D, DEV) \
            .view(n_desc, 2 * Hkv + wl.n_q_heads, D).to(torch.bfloat16)
        for i in range(n_desc):
            kn[i][0].copy_(rows[i, :Hkv]); vn[i][0].copy_(rows[i, Hkv:2 * Hkv]); qs[i][0].copy_(rows[i, 2 * Hkv:])
        qp.append_kv_layers(gb)
        qp.decode_attn_tail_layers(gb)
        torch.cuda.synchronize()
        flushed = (st + 1) // g
        assert all(gb.cache_arr[i].n_keep == wl.n_keep(i % nl) + g * flushed for i in range(n_desc))
        assert all(gb.tail_arr[i].n_tail == (st + 1) % g for i in range(n_desc))
        assert all(bool(torch.isfinite(o.float()).all()) for o in outs)
        for si, (i, hk) in enumerate(samples):
            states[si] = orc.append(states[si], bits_u16(kn[i][:, hk:hk + 1]), bits_u16(vn[i][:, hk:hk + 1]))
            if st in (0, g - 2, g - 1, g, steps - 1):
                ref = orc.decode_state(bits_u16(qs[i][:, hk * G:(hk + 1) * G]), states[si], D)
                got = outs[i][:, hk * G:(hk + 1) * G].float().cpu().numpy()
                assert np.abs(got - ref).max() <= decode_tolerance(ref), (st, i, hk)
    for si, (i, hk) in enumerate(samples):                        # the flushed group, bit for bit
        d = gb.cache_arr[i]
        n, c = d.n_keep, caches[i]
        sl = lambda t, m: t[0:1, hk:hk + 1, :m].contiguous()
        got = orc.Packed(d.bits, g, n, sl(c.k_codes, n // g).cpu().numpy().view(np.uint32),
                         sl(c.v_codes, n).cpu().numpy().view(np.uint32), bits_u16(sl(c.k_scale, n // g)),
                         bits_u16(sl(c.k_zero, n // g)), bits_u16(sl(c.v_scale, n)), bits_u16(sl(c.v_zero, n)))
        assert_packed_equal(got, states[si].packed)


def test_llama8b_compress_layers_in_the_bench_configuration():
    """qp_compress_layers over the 32 layers of an 8k sequence (the call the benchmark times) leaves, bit for bit,
    the kept indices and packed bytes of 32 qp_compress_layer calls; one sampled (layer, KV head) pair is also
    recomputed by the oracle (indices with the near-tie rule, packed bytes on the GPU's indices)."""
    wl = synth.LLAMA8B_8K
    nl, G = wl.n_layers, wl.n_q_heads // wl.n_kv_heads
    Ks, Vs, Qs = [], [], []
    for l in range(nl):
        k, v = synth.make_kv(wl, l, device=DEV)
        Ks.append(k); Vs.append(v); Qs.append(synth.make_q_win(wl, l, device=DEV))
    budgets = [wl.layer_budget_bits(l) for l in range(nl)]
    caches, kepts = qp.compress_layers(Ks, Vs, Qs, budgets, wl.bits, wl.group, wl.pool)
    torch.cuda.synchronize()
    for l in range(nl):
        ref_c, ref_k = qp.compress_layer(Ks[l], Vs[l], Qs[l], budgets[l], wl.bits, wl.group, wl.pool)
        torch.cuda.synchronize()
        assert torch.equal(kepts[l], ref_k), l
        for name in ("k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero"):
            assert torch.equal(getattr(caches[l], name), getattr(ref_c, name)), (l, name)
    layer, hk = 17, 5
    kb = bits_u16(Ks[layer][0:1, hk:hk + 1]); vb = bits_u16(Vs[layer][0:1, hk:hk + 1])
    qb = bits_u16(Qs[layer][0:1, hk * G:(hk + 1) * G])
    pooled = orc.scores(qb, kb, wl.pool)
    kept_s = kepts[layer][0:1, hk:hk + 1].cpu().numpy()
    assert check_kept_against_oracle(kept_s, pooled, wl.L, wl.w, kept_s.shape[-1]) <= 2
    assert_packed_equal(_slice_packed(caches[layer], 0, hk), orc.quantize(kb, vb, kept_s, wl.bits, wl.group))
