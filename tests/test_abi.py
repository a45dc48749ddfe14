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
    opt.use_bias = 1
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
    # option fields: biases cannot be switched off, unknown head mode / placement, a device list of the wrong length
    good = (2, 1, 64, 2, 256, 100, 1)
    for field, value in (("use_bias", 0), ("use_bias", 2), ("head_mode", 2), ("head_mode", -1), ("placement", 3),
                         ("head_layers", 65)):
        o2 = binding.il_options()
        o2.max_batch, o2.max_seq, o2.use_bias = 2, 16, 1
        setattr(o2, field, value)
        assert L.il_create(*good, C.byref(o2), C.byref(h)) == 1, (field, value)
        assert not h
    o3 = binding.il_options()
    o3.max_batch, o3.max_seq, o3.use_bias, o3.placement = 2, 16, 1, 1
    devs = (C.c_int * 3)(0, 0, 0)
    o3.devices, o3.n_devices = C.cast(devs, C.POINTER(C.c_int)), 3          # K = 2
    assert L.il_create(*good, C.byref(o3), C.byref(h)) == 1
    o3.placement, o3.n_devices = 0, 2                                        # a device list needs the pipeline placement
    assert L.il_create(*good, C.byref(o3), C.byref(h)) == 1
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


def test_operator_calls_refuse_bad_pointers_before_launching_anything():
    """Misaligned operands and sizes whose product would wrap are answered with IL_ERR_INVALID_ARG on the host
    (no device is touched: this runs without one)."""
    L = pkg.lib()
    a = 0x10000                                    # stands for a 16-byte aligned device address; never dereferenced
    assert L.il_op_attention_bwd(a, a + 2, a, a, a, a, 1, 1, 64, 2, 64, None) == 1      # o off by 2 bytes
    assert L.il_op_attention_bwd(a, a, a, a + 8, a, a, 1, 1, 64, 2, 64, None) == 1      # dout off by 8
    assert L.il_op_attention_bwd(a, a, a + 2, a, a, a, 1, 1, 64, 2, 64, None) == 1      # lse not 4-byte aligned
    assert L.il_op_attention_fwd(a, a + 4, a, 1, 64, 2, 64, None) == 1
    assert L.il_op_attention_bwd(a, a, a, a, a, a, 1, 1, 64, 2, 48, None) == 1          # unsupported head dim
    # allocation-free variant: NB * H * T = 2^64 would wrap to 0
    assert L.il_op_attention_bwd_noalloc(a, a, a, a, a, 1 << 22, 1, 1 << 21, 1 << 21, 64, None) == 1
    assert L.il_op_attention_bwd_noalloc(a, a, a, a, a, 2, 1, 1 << 20, 1, 64, None) == 1
    assert L.il_op_wait_probe(None, 10, None) == 1
    assert L.il_op_wait_probe(a, 0, None) == 1


def _expected_transfers(K, n, rule):
    """Independent statement of what crosses boundary b (between components b and b+1) backwards.
    Sum rule: one tensor per stopping level shared by the heads crossing both components.  Weighted rules: one
    tensor per head above b that component b needs — the farthest head of its window, and (unless b is the lowest
    component) every head that still has components below b to visit."""
    out = [(0, b, -1) for b in range(K - 1)]
    for b in range(K - 2, -1, -1):
        if rule == "sum":
            lv = lambda k: {max(h - n + 1, 0) for h in range(K) if max(h - n + 1, 0) <= k <= h}
            out += [(1, b, t) for t in sorted(lv(b) & lv(b + 1), reverse=True)]
        else:
            far = min(b + n - 1, K - 1)
            need = {far} if far > b else set()
            if b > 0:
                need |= {h for h in range(b + 1, K) if max(h - n + 1, 0) < b}
            need = {h for h in need if max(h - n + 1, 0) <= b < h}
            out += [(1, b, h) for h in need]
    return sorted(out)


@pytest.mark.parametrize("rule", ["sum", "far", "mean"])
@pytest.mark.parametrize("K", [1, 2, 4, 6])
def test_pipeline_transfer_plan(K, rule):
    for n in range(1, K + 1):
        plan = binding.pipeline_transfers(K, n, rule)
        assert sorted(plan) == _expected_transfers(K, n, rule), (K, n, rule)
        for b in range(K - 1):
            back = [r for r in plan if r[0] == 1 and r[1] == b]
            assert len(back) <= n - 1               # at most n-1 gradient tensors travel back per boundary
            if n == 1:
                assert not back                     # local learning: no backward communication at all (Sec. 3)
        fwd = [r for r in plan if r[0] == 0]
        assert fwd == [(0, b, -1) for b in range(K - 1)]
    with pytest.raises(binding.ILError):
        binding.pipeline_transfers(4, 5, "sum")
