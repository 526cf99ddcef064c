"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects bad arguments with status codes before launching anything."""
import ctypes
import os
import re

import pytest

from paper_2412_12706_b200 import build as qp_build
from paper_2412_12706_b200 import qp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    qp_build.build()
    return qp.lib()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "qp.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(qp_[a-z_0-9]+)\s*\(", header))
    assert declared == set(qp.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
        assert hasattr(qp, name), f"binding lacks {name}"


def test_struct_layout_matches_header():
    # 8 int32 + 4 size_t + 6 pointers
    assert ctypes.sizeof(qp.qp_cache) == 8 * 4 + 4 * 8 + 6 * 8


def test_status_strings(lib):
    seen = {qp.status_string(s) for s in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert qp.status_string(99) == "unknown status"


def test_n_keep_budget_rule():
    assert qp.n_keep(8192, 16, 32, 8192, 32) == 512
    assert qp.n_keep(8192, 8, 32, 8192, 32) == 1024
    assert qp.n_keep(8192, 4, 32, 8192, 32) == 2048
    assert qp.n_keep(16 * 5000, 16, 32, 1024, 32) == 1024
    for args, code in [((8192, 3, 32, 8192, 32), 2), ((8192, 4, 48, 8192, 32), 2), ((16 * 2, 16, 32, 1024, 32), 3),
                       ((4 * 40, 4, 32, 1024, 8), 3), ((8192, 4, 32, 8192, 8192), 1)]:
        with pytest.raises(qp.QpError) as e:
            qp.n_keep(*args)
        assert e.value.status == code


def test_cache_layout_sizes():
    c = qp.cache_layout(1, 32, 8, 128, 4, 32, 2048)
    assert c.k_codes_bytes == 8 * 2048 * 128 // 2 and c.v_codes_bytes == c.k_codes_bytes
    assert c.k_meta_bytes == 8 * 2048 * 128 // 32 * 2 and c.v_meta_bytes == c.k_meta_bytes
    total = c.k_codes_bytes + c.v_codes_bytes + 2 * c.k_meta_bytes + 2 * c.v_meta_bytes
    assert total == 2621440                           # Bt*Hkv*n*D*2*(b + 32/g)/8
    c16 = qp.cache_layout(1, 32, 8, 128, 16, 32, 1000)
    assert c16.k_codes_bytes == 8 * 1000 * 128 * 2 and c16.k_meta_bytes == 0
    for args, code in [((1, 32, 8, 128, 4, 32, 2040), 3), ((1, 32, 8, 96, 4, 32, 2048), 2),
                       ((1, 30, 8, 128, 4, 32, 2048), 1), ((1, 128, 8, 128, 4, 32, 2048), 2),
                       ((1, 32, 8, 64, 4, 128, 2048), 2)]:
        with pytest.raises(qp.QpError) as e:
            qp.cache_layout(*args)
        assert e.value.status == code


def test_tail_struct_and_capacity_layout():
    assert ctypes.sizeof(qp.qp_tail) == 2 * 4 + 2 * 8
    c = qp.cache_layout_cap(1, 32, 8, 128, 4, 32, 2048, 2048 + 256)
    assert c.n_keep == 2048 and c.n_cap == 2304
    assert c.k_codes_bytes == 8 * 2304 * 128 // 2 and c.k_meta_bytes == 8 * 2304 * 128 // 32 * 2
    assert qp.cache_layout_cap(1, 32, 8, 128, 4, 32, 2048, 0).k_codes_bytes == qp.cache_layout(1, 32, 8, 128, 4, 32, 2048).k_codes_bytes
    assert qp.cache_layout_cap(1, 32, 8, 128, 16, 32, 1000, 1001).k_codes_bytes == 8 * 1001 * 128 * 2
    # the decode workspace covers every n_keep the arrays can hold
    assert qp.decode_workspace_bytes(c) >= qp.decode_workspace_bytes(qp.cache_layout(1, 32, 8, 128, 4, 32, 2304))
    for n_cap in (2047, 2048 + 16, -32):
        with pytest.raises(qp.QpError) as e:
            qp.cache_layout_cap(1, 32, 8, 128, 4, 32, 2048, n_cap)
        assert e.value.status in (1, 3)


def test_append_and_tail_arguments_are_checked_before_any_launch(lib):
    A = 0x1000
    c = qp.cache_layout_cap(1, 8, 2, 64, 4, 32, 512, 512 + 32)
    c.k_codes = c.v_codes = c.k_scale = c.k_zero = c.v_scale = c.v_zero = A
    t = qp.qp_tail()
    t.k_tail = t.v_tail = A
    cr, tr = ctypes.byref(c), ctypes.byref(t)
    assert lib.qp_append_kv(None, A, cr, tr, None) == 1
    assert lib.qp_append_kv(A, A + 4, cr, tr, None) == 5
    assert lib.qp_append_kv(A, A, cr, None, None) == 1            # a quantized cache needs a tail
    t.n_tail = 32
    assert lib.qp_append_kv(A, A, cr, tr, None) == 1              # n_tail out of range
    t.n_tail = 31
    full = qp.cache_layout_cap(1, 8, 2, 64, 4, 32, 512, 512)
    full.k_codes = full.v_codes = full.k_scale = full.k_zero = full.v_scale = full.v_zero = A
    assert lib.qp_append_kv(A, A, ctypes.byref(full), tr, None) == 3   # the flush would not fit
    assert full.n_keep == 512 and t.n_tail == 31                  # nothing changed
    c16 = qp.cache_layout_cap(1, 8, 2, 64, 16, 32, 100, 100)
    c16.k_codes = c16.v_codes = A
    assert lib.qp_append_kv(A, A, ctypes.byref(c16), None, None) == 3
    t.n_tail = 40
    assert lib.qp_decode_attn_tail(A, cr, tr, A, A, 1 << 30, None) == 1
    t.n_tail = 3
    t.k_tail = None
    assert lib.qp_decode_attn_tail(A, cr, tr, A, A, 1 << 30, None) == 1
    t.k_tail = A + 2
    assert lib.qp_decode_attn_tail(A, cr, tr, A, A, 1 << 30, None) == 5


def test_workspace_sizes():
    assert qp.compress_workspace_bytes(1, 32, 8, 128, 8192, 32) > 8 * 8160 * 4
    assert qp.compress_workspace_bytes(1, 32, 8, 128, 32, 32) == 0
    c = qp.cache_layout(1, 32, 8, 128, 4, 32, 2048)
    # (max, sum, acc[D]) records of G heads: the larger of one per 128-token split and one per
    # (KV head + worker block), the two decompositions the decode launch can choose from
    r256 = lambda x: (x + 255) // 256 * 256
    # two areas of records (8 heads + 2432 workers) for alternate calls, or the chunked kernel's records
    assert qp.decode_workspace_bytes(c) == max(8 * (2048 // 128) * 4 * 130 * 4, 2 * r256((8 + 2432) * 4 * 130 * 4))


def test_bad_arguments_are_rejected_before_any_launch(lib):
    c = qp.cache_layout(1, 8, 2, 64, 4, 32, 512)
    A = 0x1000  # fake, aligned, never dereferenced: every call below fails validation first
    c.k_codes = c.v_codes = c.k_scale = c.k_zero = c.v_scale = c.v_zero = A
    ref = ctypes.byref(c)
    ws = 1 << 30
    call = lib.qp_compress_layer
    ok = dict(K=A, V=A, Q=A, Bt=1, Hq=8, Hkv=2, D=64, L=1024, w=32, budget=2048, bits=4, g=32, pool=7)

    def run(**kw):
        a = {**ok, **kw}
        return call(a["K"], a["V"], a["Q"], a["Bt"], a["Hq"], a["Hkv"], a["D"], a["L"], a["w"], a["budget"],
                    a["bits"], a["g"], a["pool"], ref, A, A, kw.get("ws", ws), None)

    assert run(K=None) == 1
    assert run(Hq=7) == 1
    assert run(pool=4) == 1
    assert run(w=1024) == 1
    assert run(D=96) == 2
    assert run(w=65, L=4096) == 2
    assert run(K=A + 2) == 5
    assert run(budget=16 * 8) == 3           # n <= w
    assert run(budget=2048 + 64) == 3        # cache->n_keep disagrees with the budget
    assert run(ws=16) == 4
    assert lib.qp_decode_attn(A, ref, A, A, 16, None) == 4
    assert lib.qp_decode_attn(None, ref, A, A, ws, None) == 1
    assert lib.qp_decode_attn(A + 8, ref, A, A, ws, None) == 5
    assert lib.qp_gather_quantize(A, A, None, 1024, ref, None) == 1
    assert lib.qp_select_topk(A, 1, 2, 1024, 32, 32, A, None) == 3
    assert lib.qp_window_scores(A, A, 1, 8, 2, 64, 1024, 32, 7, A, A, 16, None) == 4
    assert lib.qp_window_scores(A, A, 64, 64, 8, 64, 1 << 23, 32, 7, A, A, 1 << 62, None) == 2   # 2^32 key rows


def test_strategy_head_budget_and_overlap_arguments_are_checked_before_any_launch(lib):
    A = 0x10000
    assert ctypes.sizeof(qp.qp_side) == 2 * 4 + 4 * 8
    assert ctypes.sizeof(qp.qp_strategy) == 2 * 4 + 2 * ctypes.sizeof(qp.qp_side)
    c16 = qp.cache_layout(1, 4, 1, 128, 16, 32, 64)
    c16.k_codes = c16.v_codes = A
    s = qp.qp_strategy()
    assert lib.qp_decode_attn_ex(A, ctypes.byref(c16), ctypes.byref(s), A, A, 1 << 20, None) == 2   # nothing to quantize
    c = qp.cache_layout(1, 4, 1, 128, 4, 32, 64)
    c.k_codes = c.v_codes = c.k_scale = c.k_zero = c.v_scale = c.v_zero = A
    cr = ctypes.byref(c)
    assert lib.qp_decode_attn_ex(A, cr, None, A, A, 1 << 20, None) == 1
    s.k_axis = 2
    assert lib.qp_decode_attn_ex(A, cr, ctypes.byref(s), A, A, 1 << 20, None) == 1
    s.k_axis, s.outlier_threshold = 1, 6.0                        # filtering on, side lists missing
    assert lib.qp_gather_quantize_ex(A, A, A, 100, cr, ctypes.byref(s), None) == 1
    s.outlier_threshold = 0.0
    assert lib.qp_decode_attn_ex(A, cr, ctypes.byref(s), A, A, 16, None) == 4
    assert lib.qp_decode_attn_ex(A + 2, cr, ctypes.byref(s), A, A, 1 << 20, None) == 5

    hb = lib.qp_head_budgets
    need = lib.qp_head_budgets_workspace_bytes(2, 8, 4096, 32, 512)
    assert need >= 2 * (8 * (512 - 32) + 1) * 4 and need % 256 == 0
    assert lib.qp_head_budgets_workspace_bytes(2, 8, 4096, 32, 32) == 0
    assert hb(None, 2, 8, 4096, 32, 512, 32, A, A, need, None) == 1
    assert hb(A, 2, 8, 4096, 4096, 512, 32, A, A, need, None) == 1          # no prefix
    assert hb(A, 2, 8, 4096, 32, 512, 0, A, A, need, None) == 1
    assert hb(A, 2, 8, 4096, 32, 32, 32, A, A, need, None) == 3             # mean budget inside the window
    assert hb(A, 2, 8, 4096, 32, 512, 32, A, A + 4, need, None) == 5
    assert hb(A, 2, 8, 4096, 32, 512, 32, A, A, need - 1, None) == 4
    assert hb(A, 1, 8200, 4096, 32, 512, 32, A, A, 1 << 40, None) == 2

    words = (ctypes.c_uint32 * 4)(9, 9, 9, 9)
    assert lib.qp_debug_check(None) == 1
    assert lib.qp_debug_check(words) == 2 and list(words) == [0, 0, 0, 0]     # the release build carries no checks
