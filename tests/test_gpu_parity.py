"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, stage by stage and
end to end.  Integer, index and packed-byte results must match bit for bit; floating-point
results within the tolerances written next to each check."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import qp_oracle as orc
from paper_2412_12706_b200 import qp, synth
from tests.util import (assert_packed_equal, bf16_from_f32, bits_u16, cache_to_packed,
                        check_kept_against_oracle, decode_tolerance)

pytestmark = pytest.mark.gpu
DEV = "cuda"


def small(wl: synth.Workload, **kw) -> synth.Workload:
    return dataclasses.replace(wl, **kw)


def make_inputs(wl: synth.Workload, layer=0):
    k, v = synth.make_kv(wl, layer)
    qw = synth.make_q_win(wl, layer)
    return k, v, qw


# ------------------------------------------------------------------ S3: gather + quantize + pack

@pytest.mark.parametrize("bits", [2, 4, 8, 16])
@pytest.mark.parametrize("group,D", [(32, 128), (64, 128), (128, 128), (32, 64), (64, 64)])
def test_gather_quantize_bit_exact(bits, group, D):
    wl = small(synth.TINY, head_dim=D, n_q_heads=8, n_kv_heads=2, L=1024 + 96, batch=2)
    k, v, _ = make_inputs(wl)
    # tiny magnitudes (fp16-subnormal zero points), a constant group and exact integers
    k[0, 0, :, 5] *= 1e-6
    v[0, 1, 7, :] = 0.75
    k[1, 1, :, 9] = torch.round(k[1, 1, :, 9].float() * 4).to(torch.bfloat16)
    n = 384
    rng = np.random.default_rng(bits * 1000 + group + D)
    kept = np.stack([np.sort(rng.choice(wl.L, n, replace=False)) for _ in range(wl.batch * wl.n_kv_heads)])
    kept = kept.reshape(wl.batch, wl.n_kv_heads, n).astype(np.int32)
    ref = orc.quantize(bits_u16(k), bits_u16(v), kept, bits, group)
    cache = qp.alloc_cache(wl.batch, wl.n_q_heads, wl.n_kv_heads, D, bits, group, n, DEV)
    qp.gather_quantize(k.to(DEV), v.to(DEV), torch.from_numpy(kept).to(DEV), cache)
    torch.cuda.synchronize()
    assert_packed_equal(cache_to_packed(cache), ref)


# ------------------------------------------------------------------ S2: top-k

@pytest.mark.parametrize("P,w,n", [(992, 32, 512), (37, 5, 6), (5000, 64, 64 + 1), (4097, 8, 8 + 4096),
                                   (70000, 32, 8192), (300, 20, 320), (131072, 64, 4096 + 64),
                                   (140000, 32, 8192 + 32), (33000, 8, 8 + 1), (20000, 32, 32 + 7000)])
def test_select_topk_bit_exact_with_ties(P, w, n):
    L = P + w
    rng = np.random.default_rng(P + n)
    Bt, Hkv = 2, 3
    s = rng.random((Bt, Hkv, P)).astype(np.float32)
    s[0, 0] = np.round(s[0, 0] * 16) / 16            # heavy ties
    s[0, 1] = 0.5                                     # all equal: lowest indices win
    s[1, 0, ::3] = 0.0
    s[1, 1] = np.sort(s[1, 1])                        # ascending: the top-k is the tail
    ref = orc.select(s.astype(np.float64), L, w, n)
    got = qp.select_topk(torch.from_numpy(s).to(DEV), L, w, n)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy(), ref)


@pytest.mark.parametrize("P,w,n", [(5000, 32, 32 + 1000), (8192, 16, 16 + 4096), (20000, 32, 32 + 2048),
                                   (32736, 32, 8192), (12345, 8, 8 + 12000), (9000, 32, 32 + 1)])
@pytest.mark.parametrize("Bt,Hkv", [(4, 6), (8, 6), (16, 10)])
def test_select_topk_one_block_per_head_with_many_heads(P, w, n, Bt, Hkv):
    """With more heads than an eighth of the SMs a head is selected by one block from registers, or above 8k positions by
    a cluster of four (24 heads) or two (48 heads) while those fit in one round of the SMs, else by one block (160 heads):
    ties, constant rows, sorted rows, rows whose scores share their leading bits, denormals and zeros."""
    L = P + w
    rng = np.random.default_rng(P * 7 + n + Bt)
    s = rng.random((Bt, Hkv, P)).astype(np.float32)
    s[0, 0] = np.round(s[0, 0] * 16) / 16
    s[0, 1] = 0.5
    s[1, 0, ::3] = 0.0
    s[1, 1] = np.sort(s[1, 1])
    s[1, 2] = np.sort(s[1, 2])[::-1]
    s[2, 0] = 1.0 + rng.random(P).astype(np.float32) * 1e-4        # one leading digit, spread only in the low bits
    s[2, 1] = (rng.random(P) * 1e-40).astype(np.float32)           # denormals
    s[2, 2] = np.exp(rng.standard_normal(P) * 6).astype(np.float32)  # many binades
    s[3, 0, : P // 2] = s[3, 0, P // 2: 2 * (P // 2)]              # every value twice
    s[3, 1] = np.float32(1e-3) * (rng.integers(0, 3, P)).astype(np.float32)   # three values only
    ref = orc.select(s.astype(np.float64), L, w, n)
    got = qp.select_topk(torch.from_numpy(s).to(DEV), L, w, n)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy(), ref)


# ------------------------------------------------------------------ S1: window scores

@pytest.mark.parametrize("Hq,Hkv,D,L,w,pool", [(8, 2, 64, 1024, 32, 7), (4, 4, 128, 333, 8, 7),
                                               (16, 2, 128, 1200, 32, 5), (8, 1, 128, 700, 64, 1),
                                               (6, 2, 64, 515, 7, 3)])
def test_window_scores_close_to_oracle(Hq, Hkv, D, L, w, pool):
    wl = small(synth.TINY, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, L=L, w=w, batch=2, pool=pool)
    k, v, qw = make_inputs(wl)
    ref = orc.scores(bits_u16(qw), bits_u16(k), pool)
    got = qp.window_scores(qw.to(DEV), k.to(DEV), pool).cpu().numpy().astype(np.float64)
    rel = np.abs(got - ref) / ref
    # fp32 logits/exp against fp64: a few 1e-6 relative at worst
    assert rel.max() < 5e-6, rel.max()
    # and twice the same bits
    again = qp.window_scores(qw.to(DEV), k.to(DEV), pool).cpu().numpy()
    assert np.array_equal(again.astype(np.float64), got)


def test_window_scores_tensor_memory_path_reports_no_abandoned_wait():
    # D = 128 runs on tcgen05/TMEM; every mbarrier wait there is bounded and a block that gives up sets the
    # error word kept in the last 256 bytes of the workspace
    wl = small(synth.LLAMA8B_8K, L=4096 + 77, batch=2)
    k, v, qw = make_inputs(wl)
    nbytes = qp.compress_workspace_bytes(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.L, wl.w)
    ws = torch.full((nbytes,), 0xFF, dtype=torch.uint8, device=DEV)
    got = qp.window_scores(qw.to(DEV), k.to(DEV), wl.pool, workspace=ws).cpu().numpy().astype(np.float64)
    assert int(ws[nbytes - 256:nbytes - 252].view(torch.int32).item()) == 0
    ref = orc.scores(bits_u16(qw), bits_u16(k), wl.pool)
    assert (np.abs(got - ref) / ref).max() < 5e-6


def test_window_scores_zero_queries_closed_form():
    wl = small(synth.TINY, L=600, w=16)
    k, v, qw = make_inputs(wl)
    got = qp.window_scores(torch.zeros_like(qw).to(DEV), k.to(DEV), 1).cpu().numpy()
    G, P = wl.n_q_heads // wl.n_kv_heads, wl.L - wl.w
    u = G * sum(1.0 / (P + i + 1) for i in range(wl.w))
    assert np.allclose(got, u, rtol=2e-6)


# ------------------------------------------------------------------ S4/S5: decode attention

@pytest.mark.parametrize("bits", [2, 4, 8, 16])
@pytest.mark.parametrize("Hq,Hkv,D,group,n", [(8, 2, 64, 32, 512), (32, 8, 128, 32, 2048), (8, 8, 128, 64, 640),
                                              (16, 2, 128, 128, 1280), (4, 2, 64, 64, 192)])
def test_decode_matches_oracle(bits, Hq, Hkv, D, group, n):
    wl = small(synth.TINY, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, L=n, batch=2, group=group)
    k, v, _ = make_inputs(wl)
    kept = np.broadcast_to(np.arange(n, dtype=np.int32), (wl.batch, Hkv, n)).copy()
    pk = orc.quantize(bits_u16(k), bits_u16(v), kept, bits, group)      # oracle-made cache
    cache = qp.alloc_cache(wl.batch, Hq, Hkv, D, bits, group, n, DEV)
    qp.gather_quantize(k.to(DEV), v.to(DEV), torch.from_numpy(kept).to(DEV), cache)
    assert_packed_equal(cache_to_packed(cache), pk)
    kd, vd = orc.dequantize(pk, D)
    for step in range(2):
        q = synth.make_q_dec(wl, 0, step)
        if step == 1:
            q = (q.float() * 3).to(torch.bfloat16)        # sharper softmax
        ref = orc.decode(bits_u16(q), kd, vd)
        out = qp.decode_attn(q.to(DEV), cache).float().cpu().numpy().astype(np.float64)
        err = np.abs(out - ref).max()
        assert err <= decode_tolerance(ref), (err, decode_tolerance(ref))
        # the kernel's own budget is tighter than the stated tolerance: MMA operands (q * scale, p * scale)
        # are rounded to f16 (2^-11 relative) and the output to bf16 (2^-9 relative)
        assert err <= 3e-3 + 2.0 ** -7 * np.abs(ref).max(), err


@pytest.mark.parametrize("bits", [2, 4, 8, 16])
def test_decode_at_the_documented_magnitude_bounds(bits):
    """max|q| * max|K| just inside 2^19 and max|V| just inside 4096 (the decode calls' stated input range): the
    f16 products of the tensor-core path (query x key scale, softmax weight x value scale) stay finite and the
    result stays within the decode tolerance."""
    Hq, Hkv, D, n, group = 8, 2, 128, 1024, 32
    wl = small(synth.TINY, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, L=n, batch=1, group=group)
    k, v, _ = make_inputs(wl)
    k, v = k.float(), v.float()
    k[..., 7] *= 2000.0 / float(k[..., 7].abs().max())          # one key channel carries the large magnitudes
    v *= 4000.0 / float(v.abs().max())
    k, v = k.to(torch.bfloat16), v.to(torch.bfloat16)
    kmax = float(k.float().abs().max())
    q = synth.make_q_dec(wl, 0, 0).float()
    q[..., 7] = torch.sign(q[..., 7]) * (0.97 * 2.0 ** 19 / kmax)
    q = q.to(torch.bfloat16)
    assert float(q.float().abs().max()) * kmax <= 2.0 ** 19 and float(v.float().abs().max()) <= 4096
    kept = np.broadcast_to(np.arange(n, dtype=np.int32), (1, Hkv, n)).copy()
    pk = orc.quantize(bits_u16(k), bits_u16(v), kept, bits, group)
    cache = qp.alloc_cache(1, Hq, Hkv, D, bits, group, n, DEV)
    qp.gather_quantize(k.to(DEV), v.to(DEV), torch.from_numpy(kept).to(DEV), cache)
    assert_packed_equal(cache_to_packed(cache), pk)
    kd, vd = orc.dequantize(pk, D)
    ref = orc.decode(bits_u16(q), kd, vd)
    out = qp.decode_attn(q.to(DEV), cache).float().cpu().numpy().astype(np.float64)
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() <= decode_tolerance(ref), (np.abs(out - ref).max(), decode_tolerance(ref))


def test_decode_16bit_ragged_length_and_zero_query_mean():
    wl = small(synth.TINY, L=1000, batch=1)
    k, v, _ = make_inputs(wl)
    n = 777                                                   # not a multiple of anything
    kept = np.broadcast_to(np.arange(n, dtype=np.int32), (1, wl.n_kv_heads, n)).copy()
    cache = qp.alloc_cache(1, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, 16, 32, n, DEV)
    qp.gather_quantize(k.to(DEV), v.to(DEV), torch.from_numpy(kept).to(DEV), cache)
    q0 = torch.zeros((1, wl.n_q_heads, wl.head_dim), dtype=torch.bfloat16)
    out = qp.decode_attn(q0.to(DEV), cache).float().cpu().numpy()
    G = wl.n_q_heads // wl.n_kv_heads
    mean = v[:, :, :n].float().mean(2).numpy().repeat(G, 1)
    assert np.abs(out - mean).max() < 1e-3 + 2.0 ** -8 * np.abs(mean).max()


def test_decode_layers_equals_single_layer_calls():
    wl = small(synth.TINY, n_q_heads=8, n_kv_heads=2, head_dim=128, L=2048, batch=1)
    caches, qs, outs, singles = [], [], [], []
    for layer, n in enumerate([512, 1024, 256, 2048]):              # per-layer budgets differ
        k, v = synth.make_kv(wl, layer)
        kept = np.broadcast_to(np.arange(n, dtype=np.int32), (1, 2, n)).copy()
        c = qp.alloc_cache(1, 8, 2, 128, 4, 32, n, DEV)
        qp.gather_quantize(k.to(DEV), v.to(DEV), torch.from_numpy(kept).to(DEV), c)
        q = synth.make_q_dec(wl, layer, 0).to(DEV)
        caches.append(c); qs.append(q); outs.append(torch.empty_like(q))
        singles.append(qp.decode_attn(q, c))
    lb = qp.LayerBatch(qs, caches, outs)
    qp.decode_attn_layers(lb)
    torch.cuda.synchronize()
    for a, b in zip(outs, singles):
        # different split counts: equal up to the fp32 merge order
        assert (a.float() - b.float()).abs().max().item() <= 2.0 ** -7 * b.float().abs().max().item()


# ------------------------------------------------------------------ end to end

def run_end_to_end(wl: synth.Workload, layer=0, decode_steps=2):
    k, v, qw = make_inputs(wl, layer)
    budget = wl.layer_budget_bits(layer)
    n = orc.n_keep(budget, wl.bits, wl.group, wl.L, wl.w)
    cache, kept = qp.compress_layer(k.to(DEV), v.to(DEV), qw.to(DEV), budget, wl.bits, wl.group, wl.pool)
    torch.cuda.synchronize()
    kept_np = kept.cpu().numpy()
    assert kept_np.shape[-1] == n and n * wl.bits <= budget
    pooled = orc.scores(bits_u16(qw), bits_u16(k), wl.pool)
    swaps = check_kept_against_oracle(kept_np, pooled, wl.L, wl.w, n)
    # staged: the quantizer is checked on the GPU's own indices, so a tolerated near-tie cannot cascade
    ref = orc.quantize(bits_u16(k), bits_u16(v), kept_np, wl.bits, wl.group)
    assert_packed_equal(cache_to_packed(cache), ref)
    kd, vd = orc.dequantize(ref, wl.head_dim)
    for step in range(decode_steps):
        q = synth.make_q_dec(wl, layer, step)
        refo = orc.decode(bits_u16(q), kd, vd)
        out = qp.decode_attn(q.to(DEV), cache).float().cpu().numpy().astype(np.float64)
        assert np.abs(out - refo).max() <= decode_tolerance(refo)
    return swaps


@pytest.mark.parametrize("bits", [4, 2, 8, 16])
def test_end_to_end_tiny_config(bits):
    run_end_to_end(small(synth.TINY, bits=bits), decode_steps=16 if bits == 4 else 2)


def test_end_to_end_llama8b_8k_layer():
    swaps = run_end_to_end(synth.LLAMA8B_8K, layer=3)
    assert swaps <= 4


def test_end_to_end_pyramid_window8_group64():
    wl = small(synth.LLAMA70B_32K_B4, L=4096, batch=1, w=8, group=64, tokens16=256, n_layers=8)
    for layer in (0, 7):
        run_end_to_end(wl, layer)


def test_end_to_end_rotary_keys_2bit():
    run_end_to_end(small(synth.LLAMA8B_32K_B8, L=4096, batch=2, tokens16=256))


def test_compress_keep_all_16bit_equals_dense_attention():
    wl = small(synth.TINY, bits=16, tokens16=1024)            # budget = the whole prompt
    k, v, qw = make_inputs(wl)
    cache, kept = qp.compress_layer(k.to(DEV), v.to(DEV), qw.to(DEV), wl.budget_bits, 16)
    assert np.array_equal(kept.cpu().numpy()[0, 0], np.arange(wl.L))
    q = synth.make_q_dec(wl, 0, 0)
    out = qp.decode_attn(q.to(DEV), cache).float().cpu().numpy().astype(np.float64)
    K, V, Q = k.double().numpy(), v.double().numpy(), q.double().numpy()
    G = wl.n_q_heads // wl.n_kv_heads
    for h in range(wl.n_q_heads):
        a = K[0, h // G] @ Q[0, h] / np.sqrt(wl.head_dim)
        p = np.exp(a - a.max()); p /= p.sum()
        ref = p @ V[0, h // G]
        assert np.abs(out[0, h] - ref).max() <= 2e-3 + 2.0 ** -8 * np.abs(ref).max()


# ------------------------------------------------------------------ qp_compress_layers: many layers per launch

@pytest.mark.parametrize("bits,D,L,w", [(4, 128, 1100, 32), (2, 64, 777, 8), (16, 128, 600, 64), (8, 128, 40000, 32)])
def test_compress_layers_is_bit_identical_to_per_layer_calls(bits, D, L, w):
    """Five layers with different budgets in one qp_compress_layers call: kept indices and every packed
    byte equal those of five qp_compress_layer calls (which the other tests check against the oracle)."""
    nl, group = 5, 32
    wl = small(synth.TINY, head_dim=D, n_q_heads=8, n_kv_heads=2, L=L, w=w, batch=2, bits=bits, group=group)
    Ks, Vs, Qs = [], [], []
    for l in range(nl):
        k, v, qw = make_inputs(wl, l)
        Ks.append(k.to(DEV)); Vs.append(v.to(DEV)); Qs.append(qw.to(DEV))
    budgets = [bits * (w + 32 * (l + 1) + (0 if bits < 16 else 5)) for l in range(nl)]
    if bits < 16:
        budgets = [bits * ((w + 31) // 32 * 32 + 32 * (l + 1)) for l in range(nl)]
    caches, kepts = qp.compress_layers(Ks, Vs, Qs, budgets, bits, group, wl.pool)
    torch.cuda.synchronize()
    for l in range(nl):
        ref_c, ref_k = qp.compress_layer(Ks[l], Vs[l], Qs[l], budgets[l], bits, group, wl.pool)
        torch.cuda.synchronize()
        assert torch.equal(kepts[l], ref_k), l
        assert_packed_equal(cache_to_packed(caches[l]), cache_to_packed(ref_c))


@pytest.mark.parametrize("nl", [9, 40])
def test_compress_layers_with_many_layers_per_launch(nl):
    """The score sweeps take the layers' key tensor maps as kernel parameters in tables of 8, 32 or 128 entries: 9 and
    40 layers use the larger two.  Same comparison as above, on small layers."""
    bits, group, w = 4, 32, 16
    wl = small(synth.TINY, head_dim=64, n_q_heads=4, n_kv_heads=2, L=390, w=w, batch=1, bits=bits, group=group)
    Ks, Vs, Qs = [], [], []
    for l in range(nl):
        k, v, qw = make_inputs(wl, l)
        Ks.append(k.to(DEV)); Vs.append(v.to(DEV)); Qs.append(qw.to(DEV))
    budgets = [bits * (32 + 32 * (1 + l % 5)) for l in range(nl)]
    caches, kepts = qp.compress_layers(Ks, Vs, Qs, budgets, bits, group, wl.pool)
    torch.cuda.synchronize()
    for l in range(0, nl, 4):
        ref_c, ref_k = qp.compress_layer(Ks[l], Vs[l], Qs[l], budgets[l], bits, group, wl.pool)
        torch.cuda.synchronize()
        assert torch.equal(kepts[l], ref_k), l
        assert_packed_equal(cache_to_packed(caches[l]), cache_to_packed(ref_c))


# ------------------------------------------------------------------ per-layer token / precision mixes in one decode call

def test_decode_layers_with_mixed_precision_equals_separate_calls():
    """Sec. 5.4 swaps ranges of layers between 4 bit with 4x tokens, 8 bit with 2x and 16 bit with 1x at one budget.
    Such a mix in ONE qp_decode_attn_layers call must give, bit for bit, what a call per layer gives (and those are
    checked against the oracle above)."""
    wl = small(synth.TINY, head_dim=128, n_q_heads=8, n_kv_heads=2, L=2048 + 32, w=32, batch=2)
    budget = 16 * 256                                            # 256 tokens at 16 bit = 512 at 8 = 1024 at 4 = 2048 at 2
    plan = [(4, 32), (4, 32), (8, 32), (16, 32), (4, 64), (2, 32), (8, 32), (4, 32)]   # (bits, group) per layer
    caches, qs = [], []
    for l, (bits, group) in enumerate(plan):
        k, v, qw = make_inputs(wl, l)
        c, _ = qp.compress_layer(k.to(DEV), v.to(DEV), qw.to(DEV), budget, bits, group, wl.pool)
        assert c.desc.n_keep * bits == budget
        caches.append(c)
        qs.append(synth.make_q_dec(wl, l, 0).to(DEV))
    outs = [torch.empty_like(q) for q in qs]
    qp.decode_attn_layers(qp.LayerBatch(qs, caches, outs))
    torch.cuda.synchronize()
    for l in range(len(plan)):
        ref = qp.decode_attn(qs[l], caches[l])
        torch.cuda.synchronize()
        assert torch.equal(outs[l], ref), (l, plan[l])


# ------------------------------------------------------------------ determinism and memory hygiene

@pytest.mark.parametrize("bits", [2, 4, 8, 16])
def test_same_bits_every_run_and_no_write_outside_the_outputs(bits):
    """The whole path twice on the same inputs gives identical bytes everywhere (no floating-point atomics, fixed
    reduction orders), and guard words placed directly behind every output buffer stay untouched."""
    wl = small(synth.TINY, head_dim=128, n_q_heads=8, n_kv_heads=2, L=1500, w=32, batch=2, bits=bits,
               tokens16=384 * bits // 16)
    k, v, qw = (t.to(DEV) for t in make_inputs(wl))
    q = synth.make_q_dec(wl, 0, 0).to(DEV)
    GUARD = 64
    n = wl.n_keep(0)

    def guarded(nbytes):
        buf = torch.full((nbytes + GUARD,), 0xA5, dtype=torch.uint8, device=DEV)
        return buf

    def run():
        d = qp.cache_layout(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, bits, wl.group, n)
        sizes = [d.k_codes_bytes, d.v_codes_bytes] + ([d.k_meta_bytes] * 2 + [d.v_meta_bytes] * 2 if bits < 16 else [])
        bufs = [guarded(sz) for sz in sizes]
        d.k_codes, d.v_codes = bufs[0].data_ptr(), bufs[1].data_ptr()
        if bits < 16:
            d.k_scale, d.k_zero, d.v_scale, d.v_zero = (b.data_ptr() for b in bufs[2:])
        cache = qp.Cache(d, *bufs[:2], *(bufs[2:] if bits < 16 else [None] * 4))
        kept = guarded(wl.batch * wl.n_kv_heads * n * 4)
        out = guarded(q.numel() * 2)
        kept_t = kept[:-GUARD].view(torch.int32).view(wl.batch, wl.n_kv_heads, n)
        out_t = out[:-GUARD].view(torch.bfloat16).view_as(q)
        qp.compress_layer(k, v, qw, wl.budget_bits, bits, wl.group, wl.pool, cache, kept_t)
        qp.decode_attn(q, cache, out_t)
        torch.cuda.synchronize()
        for b in bufs + [kept, out]:
            assert bool((b[-GUARD:] == 0xA5).all()), "a kernel wrote past the end of an output buffer"
        return [b[:-GUARD].clone() for b in bufs + [kept, out]]

    first, second = run(), run()
    for a, b in zip(first, second):
        assert torch.equal(a, b)


@pytest.mark.parametrize("overlap", [False, True])
def test_calls_of_different_sizes_may_share_one_workspace(overlap):
    """Consecutive decode calls on one stream may overlap on the GPU (when enabled) and alternate between two halves
    of the workspace, whose boundary depends on the call's size: calls of different sizes on ONE workspace must still
    give the results of calls with workspaces of their own."""
    shapes = [(4, 2048), (2, 512), (8, 1024), (4, 256), (16, 512), (4, 4096)]
    caches, qs, refs = [], [], []
    for i, (bits, n) in enumerate(shapes):
        wl = small(synth.TINY, head_dim=128, n_q_heads=8, n_kv_heads=2, L=n + 300, w=32, batch=2, bits=bits,
                   tokens16=n * bits // 16)
        k, v, qw = make_inputs(wl, i)
        c, _ = qp.compress_layer(k.to(DEV), v.to(DEV), qw.to(DEV), wl.budget_bits, bits, wl.group, wl.pool)
        caches.append(c)
        qs.append(synth.make_q_dec(wl, i, 0).to(DEV))
        qp.decode_overlap(overlap)            # (a call's split over workers depends on the setting)
        refs.append(qp.decode_attn(qs[-1], c))
        torch.cuda.synchronize()
        qp.decode_overlap(False)
    ws = qp.new_decode_workspace(max(qp.decode_workspace_bytes(c) for c in caches), DEV)
    outs = [[torch.empty_like(q) for q in qs] for _ in range(5)]
    qp.decode_overlap(overlap)
    for rep in range(5):                                         # back to back, no synchronisation in between
        for i in range(len(shapes)):
            qp.decode_attn(qs[i], caches[i], outs[rep][i], ws)
    torch.cuda.synchronize()
    qp.decode_overlap(False)
    for rep in range(5):
        for i in range(len(shapes)):
            assert torch.equal(outs[rep][i], refs[i]), (rep, i, shapes[i])


# ------------------------------------------------------------------ random configurations, end to end

@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_configurations_end_to_end(seed):
    """Twelve seeded random shapes per seed (bits, head dimension, heads per group, group size, window, ragged context
    lengths, pooling width, batch, budget) through compress and decode against the oracle, stage by stage."""
    import random
    rng = random.Random(seed)
    done = 0
    while done < 12:
        bits = rng.choice([2, 4, 8, 16])
        D = rng.choice([64, 128])
        G = rng.choice([1, 2, 3, 4] if bits == 2 else [1, 2, 4, 8])
        Hkv = rng.choice([1, 2, 3])
        group = 32 if bits == 2 else rng.choice([32, 64] + ([128] if D == 128 else []))
        w = rng.choice([1, 5, 8, 16, 32, 64])
        L = rng.choice([rng.randint(300, 900), rng.randint(1000, 5000), rng.randint(5000, 9000)])
        pool = rng.choice([1, 3, 7, 13])
        batch = rng.choice([1, 2])
        unit = max(group, 32)
        n_lo, n_hi = w // unit + 1, (L - 1) // unit
        if n_hi <= n_lo:
            continue
        n = rng.randint(n_lo, min(n_hi, n_lo + 40)) * unit
        wl = small(synth.TINY, bits=bits, head_dim=D, n_q_heads=Hkv * G, n_kv_heads=Hkv, group=group, w=w, L=L,
                   pool=pool, batch=batch, tokens16=n * bits // 16, seed=synth.BASE_SEED + 7000 + 100 * seed + done)
        run_end_to_end(wl, decode_steps=2)
        done += 1


@pytest.mark.parametrize("seed", [21, 22])
def test_random_multi_layer_decode_calls(seed):
    """Eight seeded random qp_decode_attn_layers calls per seed (1 to 9 layers with their own token counts, every bit
    width, group size and heads-per-group count) against the oracle, in plain stream order and with overlapping calls:
    the flat-range split, the three merge forms and the choice between them see shapes the fixed cases do not."""
    import random
    rng = random.Random(seed)
    for case in range(8):
        bits = rng.choice([2, 4, 8, 16]); D = rng.choice([64, 128])
        G = rng.choice([1, 2, 3, 4] if bits == 2 else [1, 2, 4, 8]); Hkv = rng.choice([1, 2, 4, 8]); batch = rng.choice([1, 2, 4])
        group = 32 if bits == 2 else rng.choice([32, 64] + ([128] if D == 128 else []))
        unit = max(group, 32)
        nl = rng.choice([1, 1, 2, 3, 5, 9])
        ns = [rng.randint(1, 100 if rng.random() < 0.3 else 24) * unit for _ in range(nl)]
        wl = small(synth.TINY, n_q_heads=Hkv * G, n_kv_heads=Hkv, head_dim=D, L=max(ns), batch=batch, group=group,
                   seed=synth.BASE_SEED + 9500 + 50 * seed + case)
        caches, qs, refs = [], [], []
        for l, n in enumerate(ns):
            k, v = synth.make_kv(wl, l)
            kept = np.broadcast_to(np.arange(n, dtype=np.int32), (batch, Hkv, n)).copy()
            pk = orc.quantize(bits_u16(k), bits_u16(v), kept, bits, group)
            c = qp.alloc_cache(batch, Hkv * G, Hkv, D, bits, group, n, DEV)
            qp.gather_quantize(k.to(DEV), v.to(DEV), torch.from_numpy(kept).to(DEV), c)
            q = synth.make_q_dec(wl, l, 0)
            kd, vd = orc.dequantize(pk, D)
            refs.append(orc.decode(bits_u16(q), kd, vd)); caches.append(c); qs.append(q.to(DEV))
        for overlap in (False, True):
            outs = [torch.empty_like(x) for x in qs]
            lb = qp.LayerBatch(qs, caches, outs)
            qp.decode_overlap(overlap)
            try:
                for _ in range(3):
                    qp.decode_attn_layers(lb)
                torch.cuda.synchronize()
            finally:
                qp.decode_overlap(False)
            for l in range(nl):
                err = np.abs(outs[l].float().cpu().numpy().astype(np.float64) - refs[l]).max()
                assert err <= 3e-3 + 2.0 ** -7 * np.abs(refs[l]).max(), (case, l, ns[l], overlap, err)
