"""The allocation-free attention backward (GPU).  Some users of this library run where device allocations
are forbidden — inside another framework's memory pool, in a loop that bans cudaMalloc after start-up, under a
fixed memory budget — so il_op_attention_bwd_noalloc keeps its scratch in an array built into the library.
It must give the same gradients as il_op_attention_bwd with caller-provided scratch, call after call (the
built-in array still holds the previous call's contents), and refuse sizes beyond its fixed limit.
Collected last on purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2010_04116_b200 import binding as il

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(seed, B, T, H, dh, NB):
    g = torch.Generator(device="cpu").manual_seed(seed)
    d = H * dh
    qkv = torch.randn(B * T, 3 * d, generator=g).to(torch.bfloat16).to(DEV)
    dout = torch.randn(NB * T, d, generator=g).to(torch.bfloat16).to(DEV)
    o = torch.zeros(B * T, d, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(B, H, T, dtype=torch.float32, device=DEV)
    il.op_attention_fwd(qkv, o, lse, B, T, H, dh)
    return qkv, o, lse, dout


def test_no_alloc_attention_backward_matches_on_two_calls_in_a_row():
    # two different problems back to back: the second call finds the first call's values in the shared scratch
    for seed, (B, T, H, dh, NB) in enumerate([(2, 200, 3, 64, 4), (1, 130, 2, 80, 1)]):
        qkv, o, lse, dout = _case(seed, B, T, H, dh, NB)
        d = H * dh
        ref = torch.zeros(NB * T, 3 * d, dtype=torch.bfloat16, device=DEV)
        delta = torch.zeros(NB * H * T, dtype=torch.float32, device=DEV)
        il.op_attention_bwd(qkv, o, lse, dout, ref, delta, NB, B, T, H, dh)
        got = torch.full((NB * T, 3 * d), 7.0, dtype=torch.bfloat16, device=DEV)
        before = torch.cuda.memory_allocated()
        il.op_attention_bwd_noalloc(qkv, o, lse, dout, got, NB, B, T, H, dh)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        a, b = got.float().cpu().numpy(), ref.float().cpu().numpy()
        assert np.isfinite(a).all()
        rel = np.linalg.norm(a - b) / np.linalg.norm(b)
        assert rel < 1.5e-2, rel          # tolerance of the attention parity tests; the two paths are in fact identical
        assert np.array_equal(a, b)
        assert il.op_attention_bwd_noalloc_status() == 0      # no bounded wait expired in that call
        # and directly against the fp64 oracle's attention backward (first gradient batch)
        from oracle import il_oracle as orc
        ref64 = orc.attention_bwd(dout[:B * T].float().cpu().numpy().astype(np.float64),
                                  qkv.float().cpu().numpy().astype(np.float64), B, T, H)
        rel64 = np.linalg.norm(a[:B * T] - ref64) / np.linalg.norm(ref64)
        assert rel64 < 1.5e-2, rel64


def test_no_alloc_attention_backward_rejects_sizes_beyond_its_scratch():
    limit = il.lib().il_op_attention_bwd_noalloc_max_rows()
    assert limit == 1 << 20
    t = torch.zeros(8, dtype=torch.float32, device=DEV)
    with pytest.raises(il.ILError) as e:     # NB*H*T = 2 * limit: refused on the host, nothing is launched
        il.op_attention_bwd_noalloc(t, t, t, t, t, 2, 1, int(limit), 1, 64)
    assert e.value.status == 1
    torch.cuda.synchronize()
