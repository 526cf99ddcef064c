"""qp_decode_attn_static: the decode entry point for hosts that cannot allocate scratch.

Collected last on purpose (file name), so a run that stops at the first failure has already
gone through every other test.  Checks, through the C ABI, that the built-in-scratch variant
returns what qp_decode_attn returns with a caller workspace, on two calls in a row that share
the scratch array, and that an oversized request is refused before anything is launched.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2412_12706_b200 import qp, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _cache(wl, n, bits):
    k, v = synth.make_kv(wl, 0)
    kept = torch.arange(n, dtype=torch.int32).expand(wl.batch, wl.n_kv_heads, n).contiguous()
    c = qp.alloc_cache(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, bits, wl.group, n, DEV)
    qp.gather_quantize(k.to(DEV), v.to(DEV), kept.to(DEV), c)
    return c


def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    wl = synth.dataclasses.replace(synth.TINY, n_q_heads=32, n_kv_heads=8, head_dim=128, L=2048, batch=2)
    big, small = _cache(wl, 2048, 4), _cache(wl, 640, 2)
    # two back-to-back calls that reuse the shared array, the second with a different cache shape
    for step, cache in enumerate((big, small, big)):
        q = synth.make_q_dec(wl, 0, step).to(DEV)
        ref = qp.decode_attn(q, cache)
        got = qp.decode_attn_static(q, cache)
        torch.cuda.synchronize()
        r, g = ref.float().cpu().numpy(), got.float().cpu().numpy()
        # same kernels, same split: the tolerance of the decode tests is more than needed
        assert np.abs(g - r).max() <= 1e-2 + 1e-2 * np.abs(r).max()
        assert np.array_equal(g, r)


def test_static_scratch_rejects_oversized_cache_without_launching():
    # 8 query heads per KV head at 2 bits take the chunked kernel, whose scratch is one record per
    # (batch x KV head, token split, query head of the group):
    # 1024 (batch x KV head) pairs x 2 splits x 8 heads x 130 floats = 8.5 MB > 4 MiB
    c = qp.cache_layout(128, 64, 8, 128, 2, 32, 4096)
    fake = 0x10000   # aligned, never dereferenced: the size check comes before any launch
    c.k_codes = c.v_codes = c.k_scale = c.k_zero = c.v_scale = c.v_zero = fake
    st = qp.lib().qp_decode_attn_static(fake, ctypes.byref(c), fake, None)
    assert st == 4
    torch.cuda.synchronize()       # the context is still healthy
    with pytest.raises(qp.QpError):
        qp.decode_attn_static(torch.zeros((1, 8, 64), dtype=torch.bfloat16, device=DEV),
                              type("C", (), {"desc": c})())
