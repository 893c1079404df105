"""The C-ABI library loads, exports every symbol the header declares, and its size queries and
argument checks behave without a GPU."""
import ctypes as C
import os
import re

import pytest

import paper_2605_08696_b200 as P
from paper_2605_08696_b200 import binding as Bd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _header_functions():
    txt = open(os.path.join(ROOT, "include", "srm.h")).read()
    txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
    return sorted(set(re.findall(r"\b(srm_[a-z_0-9]+)\s*\(", txt)))


def test_every_declared_symbol_is_exported_and_bound():
    lib = P.load_library()
    names = _header_functions()
    assert len(names) >= 25
    for n in names:
        assert hasattr(lib, n), f"{n} declared in srm.h but not exported"
        assert n in Bd.SYMBOLS, f"{n} has no ctypes signature in the binding"
    assert sorted(Bd.SYMBOLS) == names


def _cfg(**kw):
    base = dict(n_layers=2, d_model=64, n_heads=4, ffn_mult=4, vocab=256, n_ctx=32, dtype=0, state_dtype=0,
                ln_eps=1e-5, flags=0, mixer=0, kernel_size=1)
    base.update(kw)
    return Bd._Config(*[base[k] for k, _ in Bd._Config._fields_])


def test_size_queries_and_layout():
    lib = P.load_library()
    c = _cfg()
    total = lib.srm_weights_bytes(C.byref(c))
    assert total > 0 and total % 256 == 0
    # slots are disjoint, ordered, 256-aligned and cover what the shapes say
    seen = []
    for layer, tids in [(-1, [0, 12, 13, 14])] + [(l, list(range(1, 12))) for l in range(2)]:
        for t in tids:
            off, nb, eb = C.c_size_t(), C.c_size_t(), C.c_int32()
            assert lib.srm_weight_slot(C.byref(c), layer, t, C.byref(off), C.byref(nb), C.byref(eb)) == 0
            assert off.value % 256 == 0 and off.value + nb.value <= total
            seen.append((off.value, nb.value))
    seen.sort()
    for (o1, n1), (o2, _) in zip(seen, seen[1:]):
        assert o1 + n1 <= o2
    V, d, F, n, h = 256, 64, 256, 32, 4
    params = 2 * V * d + 2 * d + 2 * (4 * d + h * n + n * d + h + 2 * F * d + F + d)
    assert sum(nb for _, nb in seen) == 4 * params
    # bf16 halves the matrices only
    cb = _cfg(dtype=1)
    assert lib.srm_weights_bytes(C.byref(cb)) < total
    # state: one d-vector per layer per sample (+ header and last-token vector)
    s1, s2 = lib.srm_state_bytes(C.byref(c), 1000), lib.srm_state_bytes(C.byref(c), 2000)
    # cache rows + last-token, position and top-k threshold vectors (4000 -> 4096, 8000 -> 8192 bytes each)
    assert s2 - s1 == 1000 * (2 * 64 * 4) + 3 * 4096
    assert lib.srm_workspace_bytes(C.byref(c), 8, 0) < lib.srm_workspace_bytes(C.byref(c), 16, 0)


@pytest.mark.parametrize("bad", [dict(d_model=100), dict(n_heads=3), dict(vocab=250), dict(n_layers=0),
                                 dict(dtype=7), dict(d_model=4096), dict(ln_eps=0.0)])
def test_invalid_configs_are_rejected(bad):
    lib = P.load_library()
    c = _cfg(**bad)
    assert lib.srm_weights_bytes(C.byref(c)) == 0
    assert lib.srm_state_bytes(C.byref(c), 4) == 0
    out = C.c_void_p()
    fake = C.c_void_p(256)
    assert lib.srm_create(C.byref(c), fake, 1 << 30, C.byref(out)) == -2   # SRM_ERR_UNSUPPORTED
    assert not out.value


def test_null_and_alignment_errors_without_device_work():
    lib = P.load_library()
    c = _cfg()
    out = C.c_void_p()
    assert lib.srm_create(C.byref(c), None, 0, C.byref(out)) == -1
    assert lib.srm_create(C.byref(c), C.c_void_p(8), 1 << 30, C.byref(out)) == -3
    assert lib.srm_create(C.byref(c), C.c_void_p(256), 16, C.byref(out)) == -4
    assert lib.srm_decode_step(None, None, None, None, 0, None, None, None, 0, None) == -1
    assert lib.srm_strerror(-5) == b"position would exceed n_ctx"
    assert lib.srm_state_pos(None) == -1


def test_decode_pass_rows_rule():
    """Small batches run as one pass, large ones as equal passes of whole 256-row tiles of at most 10240 rows,
    and a small workspace decides by itself. Every pass size is positive and the passes cover the batch."""
    lib = P.load_library()
    f = lib.srm_decode_pass_rows
    assert f(0, 100) == 0 and f(100, 0) == 0
    assert f(1, 1 << 20) == 1 and f(4096, 1 << 20) == 4096 and f(12288, 1 << 20) == 12288
    assert f(16384, 1 << 20) == 8192 and f(32768, 1 << 20) == 8192 and f(37888, 1 << 20) == 9472
    assert f(20000, 1 << 20) == 10240                      # two passes: 10240 + 9760
    assert f(12289, 1 << 20) == 6400                       # two passes of 25 tiles
    assert f(4096, 1000) == 1000 and f(100000, 8192) == 8192 and f(100000, 300) == 300
    assert f(8192, 8192) == 8192 and f(8192, 8191) == 8191
    assert f(1 << 21, 49152) == 10240
    for B in (1, 255, 6145, 12288, 12289, 16385, 99999, 1 << 21):
        for fit in (1, 255, 4096, 10239, 10240, 16384, 1 << 22):
            r = f(B, fit)
            assert 1 <= r <= min(B, fit), (B, fit, r)
            if B > 12288 and fit >= 10240:
                assert r % 256 == 0 and r <= 10240
