"""The range-checked debug build (libqp_checked.so): the whole path on valid inputs records no violation, and the
normal build reports that it has no checks.  Runs in a child process because a process loads one build of the
library.  No test feeds the GPU an out-of-range index: the checked build exists to find such bugs, not to be
driven into them."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import dataclasses, sys
import numpy as np, torch
sys.path.insert(0, %(root)r)
from paper_2412_12706_b200 import qp, synth
dev = "cuda"
st, w = qp.debug_check()
assert st == %(want_status)d, (st, w)
for bits, group, k_axis, thr in [(4, 32, 0, None), (2, 32, 1, 6.0), (8, 64, 0, 6.0), (16, 32, 0, None)]:
    wl = dataclasses.replace(synth.TINY, bits=bits, group=group, tokens16=512 * bits // 16, head_dim=128, L=1500, batch=2)
    k, v = synth.make_kv(wl, 0); qw = synth.make_q_win(wl, 0)
    cache, kept = qp.compress_layer(k.to(dev), v.to(dev), qw.to(dev), wl.budget_bits, bits, group, wl.pool,
                                    n_cap=wl.n_keep(0) + 2 * group)
    q = synth.make_q_dec(wl, 0, 0).to(dev)
    out = qp.decode_attn(q, cache)
    tail = qp.alloc_tail(cache)
    for s in range(group + 3):
        kn, vn = synth.make_kv_new(wl, 0, s)
        qp.append_kv(kn.to(dev), vn.to(dev), cache, tail)
        qp.decode_attn_tail(q, cache, tail)
    if bits < 16:
        c2 = qp.alloc_cache(wl.batch, wl.n_q_heads, wl.n_kv_heads, 128, bits, group, wl.n_keep(0), dev)
        strat = qp.make_strategy(c2, k_axis, thr)
        qp.gather_quantize_ex(k.to(dev), v.to(dev), kept, c2, strat)
        qp.decode_attn_ex(q, c2, strat)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
st, w = qp.debug_check()
assert st == %(want_status)d and w == [0, 0, 0, 0], (st, w)
print("CHECKED-OK")
"""


@pytest.mark.parametrize("lib,want_status", [("libqp_checked.so", 0), ("libqp.so", 2)])
def test_whole_path_on_valid_inputs_records_no_violation(lib, want_status):
    path = os.path.join(ROOT, "paper_2412_12706_b200", lib)
    assert os.path.exists(path), "build it with python -m paper_2412_12706_b200.build"
    env = dict(os.environ, QP_LIBRARY=path)
    res = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT, "want_status": want_status}], env=env,
                         capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and "CHECKED-OK" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]
