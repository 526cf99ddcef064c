"""Consecutive decode calls that are allowed to overlap on the GPU (qp_decode_overlap) must give, bit for
bit, the results of calls that run one after the other.

The cases here are the ones where an ordering mistake would show as wrong numbers: many small launches
(a handful of blocks each, so that several kernels fit on the GPU at once) replayed back to back from a
CUDA graph on ONE workspace, with a different query and output per call.  Nothing in these tests waits
on the GPU or expects a fault: they only compare outputs.
"""
import dataclasses

import pytest
import torch

from paper_2412_12706_b200 import qp, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _layers(bits, n_caches, n_tokens, G=4):
    """A few small single-layer caches (Llama-like heads, batch 1) and their descriptors."""
    caches = []
    wl = dataclasses.replace(synth.TINY, head_dim=128, n_kv_heads=8, n_q_heads=8 * G, L=n_tokens + 200, w=32,
                             batch=1, bits=bits, tokens16=n_tokens * bits // 16)
    for i in range(n_caches):
        k, v = synth.make_kv(wl, i)
        qw = synth.make_q_win(wl, i)
        c, _ = qp.compress_layer(k.to(DEV), v.to(DEV), qw.to(DEV), wl.budget_bits, bits, wl.group, wl.pool)
        caches.append(c)
    torch.cuda.synchronize()
    return wl, caches


def _separated(call, n_calls, overlap_setting):
    """Reference: every call followed by a synchronisation, so nothing can overlap.  The stream's overlap setting
    is the one under test, because the split of a call over workers (and with it the last bits of the result)
    depends on the setting; results are bit-reproducible within a setting."""
    outs = []
    qp.decode_overlap(overlap_setting)
    for i in range(n_calls):
        outs.append(call(i))
        torch.cuda.synchronize()
    qp.decode_overlap(False)
    return outs


@pytest.mark.parametrize("bits,n_tokens", [(4, 2048), (2, 2048), (8, 1024), (16, 512), (4, 256)])
def test_graph_replay_of_a_chain_of_small_calls_on_one_workspace(bits, n_tokens):
    n_calls, n_caches, reps = 96, 6, 5
    wl, caches = _layers(bits, n_caches, n_tokens)
    qs = [synth.make_q_dec(wl, i % n_caches, i).to(DEV) for i in range(n_calls)]
    ws = qp.new_decode_workspace(max(qp.decode_workspace_bytes(c) for c in caches), DEV)
    refs = _separated(lambda i: qp.decode_attn(qs[i], caches[i % n_caches]), n_calls, True)
    refs_off = _separated(lambda i: qp.decode_attn(qs[i], caches[i % n_caches]), n_calls, False)

    outs = [torch.zeros_like(q) for q in qs]
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        qp.decode_overlap(True)                                   # for this stream only
        qp.decode_attn(qs[0], caches[0], outs[0], ws)             # warm-up outside the capture
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            for i in range(n_calls):
                qp.decode_attn(qs[i], caches[i % n_caches], outs[i], ws)
        for rep in range(reps):
            for o in outs:
                o.zero_()
            graph.replay()
            graph.replay()                                        # two replays back to back overlap as well
            side.synchronize()
            for i in range(n_calls):
                assert torch.equal(outs[i], refs[i]), (rep, i)
        # the same chain issued directly (not from a graph), and with the overlap switched off again
        for on in (True, False):
            qp.decode_overlap(on)
            for o in outs:
                o.zero_()
            for i in range(n_calls):
                qp.decode_attn(qs[i], caches[i % n_caches], outs[i], ws)
            side.synchronize()
            for i in range(n_calls):
                assert torch.equal(outs[i], (refs if on else refs_off)[i]), (on, i)


def test_graph_replay_through_the_built_in_scratch():
    n_calls, n_caches = 64, 4
    wl, caches = _layers(4, n_caches, 1024)
    qs = [synth.make_q_dec(wl, i % n_caches, 100 + i).to(DEV) for i in range(n_calls)]
    refs = _separated(lambda i: qp.decode_attn(qs[i], caches[i % n_caches]), n_calls, True)
    outs = [torch.zeros_like(q) for q in qs]
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        qp.decode_overlap(True)
        qp.decode_attn_static(qs[0], caches[0], outs[0])          # the first call on a device: outside any capture
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            for i in range(n_calls):
                qp.decode_attn_static(qs[i], caches[i % n_caches], outs[i])
        for rep in range(3):
            for o in outs:
                o.zero_()
            graph.replay()
            side.synchronize()
            for i in range(n_calls):
                assert torch.equal(outs[i], refs[i]), (rep, i)
        qp.decode_overlap(False)


def test_a_call_that_reads_the_previous_output_is_not_started_early():
    """q of call i+1 is the out buffer of call i: the library must notice and keep stream order."""
    wl, caches = _layers(4, 2, 1024)
    n_calls = 24
    q0 = synth.make_q_dec(wl, 0, 7).to(DEV)
    bufs = [q0] + [torch.zeros_like(q0) for _ in range(n_calls)]
    ref = [q0]
    qp.decode_overlap(True)
    for i in range(n_calls):
        ref.append(qp.decode_attn(ref[-1], caches[i % 2]))
        torch.cuda.synchronize()
    qp.decode_overlap(False)
    ws = qp.new_decode_workspace(qp.decode_workspace_bytes(caches[0]), DEV)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        qp.decode_overlap(True)
        for rep in range(3):
            for i in range(n_calls):
                qp.decode_attn(bufs[i], caches[i % 2], bufs[i + 1], ws)
            side.synchronize()
            for i in range(n_calls):
                assert torch.equal(bufs[i + 1], ref[i + 1]), (rep, i)
        qp.decode_overlap(False)


@pytest.mark.parametrize("bits", [4, 2])
def test_generation_loop_with_overlap_matches_the_loop_without(bits):
    """append + attention-with-tail for many steps with the overlap enabled: issued back to back, against the same
    loop with a synchronisation after every step."""
    group, steps = 32, 2 * 32 + 9
    wl = dataclasses.replace(synth.TINY, head_dim=128, n_kv_heads=8, n_q_heads=32, L=1500, w=32, batch=1, bits=bits,
                             tokens16=1024 * bits // 16)
    k, v = synth.make_kv(wl, 0)
    qw = synth.make_q_win(wl, 0)
    kd, vd, qwd = k.to(DEV), v.to(DEV), qw.to(DEV)
    news = [tuple(t.to(DEV) for t in synth.make_kv_new(wl, 0, s)) for s in range(steps)]
    qs = [synth.make_q_dec(wl, 0, s).to(DEV) for s in range(steps)]
    results = []
    side = torch.cuda.Stream()
    for back_to_back in (False, True):
        with torch.cuda.stream(side):
            qp.decode_overlap(True)
            cache, _ = qp.compress_layer(kd, vd, qwd, wl.budget_bits, bits, group, wl.pool,
                                         n_cap=wl.n_keep(0) + 3 * group)
            tail = qp.alloc_tail(cache)
            ws = qp.new_decode_workspace(qp.decode_workspace_bytes(cache), DEV)
            outs = [torch.zeros_like(q) for q in qs]
            for s in range(steps):
                qp.append_kv(news[s][0], news[s][1], cache, tail)
                qp.decode_attn_tail(qs[s], cache, tail, outs[s], ws)
                if not back_to_back:
                    side.synchronize()
            side.synchronize()
            qp.decode_overlap(False)
        results.append(outs)
    for s in range(steps):
        assert torch.equal(results[0][s], results[1][s]), s
