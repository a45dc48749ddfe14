"""CPU-side checks of the C-ABI library: it loads, exports every symbol the headers declare, and its
host-only logic (argument validation that needs no device, the n-wise stream bookkeeping) is right."""
import ctypes as C
import os
import re

import pytest

import paper_2010_04116_b200 as pkg
from paper_2010_04116_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    for h in ("il.h", "il_ops.h"):
        src = open(os.path.join(ROOT, "include", h)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names |= set(re.findall(r"\b(il_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_library_loads_and_exports_every_declared_symbol():
    L = pkg.lib()
    syms = _declared_symbols()
    assert len(syms) >= 25
    for s in syms:
        assert hasattr(L, s), s


def test_status_strings():
    L = pkg.lib()
    assert L.il_status_string(0) == b"IL_OK"
    assert L.il_status_string(5) == b"IL_ERR_TIMEOUT"


def test_create_rejects_bad_arguments_without_a_device():
    L = pkg.lib()
    h = C.c_void_p(None)
    opt = binding.il_options()
    opt.max_batch, opt.max_seq = 2, 16
    bad = [
        (2, 1, 64, 2, 256, 100, 3),     # n > K
        (2, 1, 64, 2, 256, 100, 0),     # n < 1
        (2, 1, 60, 2, 256, 100, 1),     # d % 8
        (2, 1, 64, 3, 256, 100, 1),     # d % H
        (2, 1, 64, 4, 256, 100, 1),     # head dim 16 unsupported
        (0, 1, 64, 2, 256, 100, 1),     # K < 1
    ]
    for a in bad:
        assert L.il_create(*a, C.byref(opt), C.byref(h)) == 1, a
        assert not h
    assert L.il_create(2, 1, 64, 2, 256, 100, 1, None, C.byref(h)) == 1
    assert L.il_create(2, 1, 64, 2, 256, 100, 1, C.byref(opt), None) == 1
    assert L.il_sync(None) == 1
    assert L.il_num_tensors(None) == -1


def _expected_streams(K, n, k):
    """Independent statement: heads crossing component k, grouped by where their gradient stops."""
    heads = [h for h in range(K) if max(h - n + 1, 0) <= k <= h]
    return sorted({max(h - n + 1, 0) for h in heads}, reverse=True)


@pytest.mark.parametrize("K", [1, 2, 4, 8])
def test_nwise_stream_bookkeeping(K):
    for n in range(1, K + 1):
        counts = []
        for k in range(K):
            t = pkg.nwise_streams(K, n, k)
            assert t == _expected_streams(K, n, k)
            counts.append(len(t))
            # closed form for the number of stacked backward passes of component k+1 (1-based kk)
            kk = k + 1
            s = 1 + max(0, min(kk + n - 1, K) - n) if kk <= n else min(kk + n - 1, K) - kk + 1
            assert len(t) == s
        if n == 1 or n == K:
            assert counts == [1] * K      # local learning / ordinary backprop: one pass per component
    with pytest.raises(binding.ILError):
        pkg.nwise_streams(4, 5, 0)
    assert [len(pkg.nwise_streams(8, 2, k)) for k in range(8)] == [1, 2, 2, 2, 2, 2, 2, 1]
    assert [len(pkg.nwise_streams(8, 3, k)) for k in range(8)] == [1, 2, 3, 3, 3, 3, 2, 1]
