"""GPU parity of the decode-time append path (Eq. 2 on the quantized-pruned cache): rows appended
through the C ABI, attention over packed tokens plus tail, and the quantization of full tails,
against the CPU oracle.  Packed bytes must match bit for bit, outputs within the decode tolerance."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import qp_oracle as orc
from paper_2412_12706_b200 import qp, synth
from tests.util import assert_packed_equal, bits_u16, cache_to_packed, decode_tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda"


def workload(bits, group, D, G, **kw):
    base = dict(head_dim=D, n_kv_heads=2, n_q_heads=2 * G, L=640, w=32, batch=2, bits=bits, group=group,
                tokens16=256 * bits // 16)                        # n_keep = 256 tokens at every width
    base.update(kw)
    return dataclasses.replace(synth.TINY, **base)


def compress(wl, n_cap_extra):
    k, v = synth.make_kv(wl, 0)
    qw = synth.make_q_win(wl, 0)
    n = wl.n_keep(0)
    cache, _ = qp.compress_layer(k.to(DEV), v.to(DEV), qw.to(DEV), wl.budget_bits, wl.bits, wl.group, wl.pool,
                                 n_cap=n + n_cap_extra if n_cap_extra else 0)
    torch.cuda.synchronize()
    return cache


# (bits, group, D, G): all four tensor-core kernels, groups of 64 / 128, and shapes that take the generic kernel
SHAPES = [(4, 32, 128, 4), (4, 64, 128, 4), (4, 128, 128, 2), (4, 32, 64, 4), (8, 32, 128, 4), (8, 64, 128, 8),
          (2, 32, 128, 4), (2, 32, 128, 8), (2, 64, 128, 4), (16, 32, 128, 4), (16, 32, 64, 8),
          (4, 32, 64, 3), (8, 32, 128, 1), (2, 32, 128, 3)]      # odd group sizes: a merge block's second warp may idle


@pytest.mark.parametrize("bits,group,D,G", SHAPES)
def test_generation_loop_matches_oracle(bits, group, D, G):
    wl = workload(bits, group, D, G)
    steps = 2 * group + 5 if bits < 16 else 37
    cache = compress(wl, 3 * group)
    tail = qp.alloc_tail(cache)
    n0 = cache.desc.n_keep
    st = orc.gen_state(cache_to_packed(cache), D)                # the oracle starts from the GPU's own prompt cache
    ws = qp.new_decode_workspace(qp.decode_workspace_bytes(cache), DEV)
    worst = 0.0
    for s in range(steps):
        kn, vn = synth.make_kv_new(wl, 0, s)
        qp.append_kv(kn.to(DEV), vn.to(DEV), cache, tail)
        st = orc.append(st, bits_u16(kn), bits_u16(vn))
        assert cache.desc.n_keep == st.packed.n and tail.desc.n_tail == st.n_tail
        q = synth.make_q_dec(wl, 0, s)
        out = qp.decode_attn_tail(q.to(DEV), cache, tail, workspace=ws)
        torch.cuda.synchronize()
        ref = orc.decode_state(bits_u16(q), st, D)
        err = float(np.abs(out.float().cpu().numpy() - ref).max())
        assert err <= decode_tolerance(ref), (s, err)
        worst = max(worst, err)
    assert cache.desc.n_keep == (n0 + 2 * group if bits < 16 else n0 + steps)
    assert_packed_equal(cache_to_packed(cache), st.packed)       # flushed groups bit-exact, old ones untouched
    if bits < 16 and st.n_tail:
        assert np.array_equal(bits_u16(tail.k_tail)[:, :, :st.n_tail], st.tail_k)
        assert np.array_equal(bits_u16(tail.v_tail)[:, :, :st.n_tail], st.tail_v)


@pytest.mark.parametrize("bits,group,D,G", [(4, 32, 128, 4), (8, 128, 128, 4), (2, 32, 128, 4), (2, 64, 128, 4),
                                            (16, 32, 128, 4)])
def test_room_for_appends_does_not_change_the_result(bits, group, D, G):
    """A cache with spare capacity holds the same bytes and decodes to the same bits as a tight one."""
    wl = workload(bits, group, D, G)
    tight, roomy = compress(wl, 0), compress(wl, 5 * group)
    assert roomy.desc.n_cap == tight.desc.n_keep + 5 * group and roomy.nbytes > tight.nbytes
    assert_packed_equal(cache_to_packed(roomy), cache_to_packed(tight))
    q = synth.make_q_dec(wl, 0, 0).to(DEV)
    a, b = qp.decode_attn(q, tight), qp.decode_attn(q, roomy)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    tail = qp.alloc_tail(roomy)                                   # an empty tail changes nothing either
    c = qp.decode_attn_tail(q, roomy, tail)
    torch.cuda.synchronize()
    assert torch.equal(a, c)


def test_append_without_room_is_refused_and_changes_nothing():
    wl = workload(4, 32, 128, 4)
    cache = compress(wl, 32)
    tail = qp.alloc_tail(cache)
    kn, vn = (t.to(DEV) for t in synth.make_kv_new(wl, 0, 0))
    for _ in range(32 + 31):
        qp.append_kv(kn, vn, cache, tail)
    assert cache.desc.n_keep == wl.n_keep(0) + 32 and tail.desc.n_tail == 31
    with pytest.raises(qp.QpError) as e:
        qp.append_kv(kn, vn, cache, tail)
    assert e.value.status == 3 and cache.desc.n_keep == wl.n_keep(0) + 32 and tail.desc.n_tail == 31
    torch.cuda.synchronize()


@pytest.mark.parametrize("bits", [4, 16])
def test_layers_calls_with_layers_in_different_states(bits):
    """qp_append_kv_layers / qp_decode_attn_tail_layers over three layers whose tails hold different numbers of
    tokens (so that they flush on different steps) and whose caches differ in n_keep."""
    group, D, G, nl = 32, 128, 4, 3
    wls = [workload(bits, group, D, G, tokens16=(256 + 64 * l) * bits // 16, seed=synth.BASE_SEED + 50 + l)
           for l in range(nl)]
    caches = [compress(w, 4 * group) for w in wls]
    tails = [qp.alloc_tail(c) for c in caches]
    states = [orc.gen_state(cache_to_packed(c), D) for c in caches]
    for l in range(nl):                                          # stagger: layer l starts with 9*l tail tokens
        for s in range(9 * l):
            kn, vn = synth.make_kv_new(wls[l], 0, 1000 + s)
            qp.append_kv(kn.to(DEV), vn.to(DEV), caches[l], tails[l])
            states[l] = orc.append(states[l], bits_u16(kn), bits_u16(vn))
    mk = lambda: [torch.empty((2, 2, D), dtype=torch.bfloat16, device=DEV) for _ in range(nl)]
    kns, vns = mk(), mk()
    qs = [torch.empty((2, 2 * G, D), dtype=torch.bfloat16, device=DEV) for _ in range(nl)]
    outs = [torch.empty_like(q) for q in qs]
    gb = qp.GenBatch(qs, kns, vns, caches, tails, outs)
    for s in range(40):
        for l in range(nl):
            kn, vn = synth.make_kv_new(wls[l], 0, s)
            kns[l].copy_(kn); vns[l].copy_(vn)
            qs[l].copy_(synth.make_q_dec(wls[l], 0, s))
            states[l] = orc.append(states[l], bits_u16(kn), bits_u16(vn))
        qp.append_kv_layers(gb)
        qp.decode_attn_tail_layers(gb)
        torch.cuda.synchronize()
        for l in range(nl):
            assert gb.cache_arr[l].n_keep == states[l].packed.n and gb.tail_arr[l].n_tail == states[l].n_tail
            ref = orc.decode_state(bits_u16(qs[l]), states[l], D)
            err = float(np.abs(outs[l].float().cpu().numpy() - ref).max())
            assert err <= decode_tolerance(ref), (s, l, err)
    for l in range(nl):
        assert_packed_equal(cache_to_packed(caches[l], gb.cache_arr[l]), states[l].packed)


@pytest.mark.parametrize("bits,n", [(4, 4096), (8, 2080), (2, 3104)])
def test_generation_steps_on_a_long_cache_with_many_records_per_row(bits, n):
    """One layer with thousands of kept tokens leaves dozens of partial records per output row; the merge that also
    folds the tail takes them four at a time (the last batch is ragged for these sizes)."""
    group, D, G = 32, 128, 4
    wl = workload(bits, group, D, G, L=n + 1500, tokens16=n * bits // 16, batch=1)
    cache = compress(wl, 2 * group)
    tail = qp.alloc_tail(cache)
    st = orc.gen_state(cache_to_packed(cache), D)
    ws = qp.new_decode_workspace(qp.decode_workspace_bytes(cache), DEV)
    for s in range(group + 3):
        kn, vn = synth.make_kv_new(wl, 0, s)
        qp.append_kv(kn.to(DEV), vn.to(DEV), cache, tail)
        st = orc.append(st, bits_u16(kn), bits_u16(vn))
        if s % 7 and s < group:
            continue
        q = synth.make_q_dec(wl, 0, s)
        out = qp.decode_attn_tail(q.to(DEV), cache, tail, workspace=ws)
        torch.cuda.synchronize()
        ref = orc.decode_state(bits_u16(q), st, D)
        err = float(np.abs(out.float().cpu().numpy() - ref).max())
        assert err <= decode_tolerance(ref), (s, err)
        assert err <= 3e-3 + 2.0 ** -7 * float(np.abs(ref).max()), (s, err)
    assert_packed_equal(cache_to_packed(cache), st.packed)
