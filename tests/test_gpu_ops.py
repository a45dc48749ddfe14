"""Operator-level parity (GPU): each CUDA kernel, called through the C ABI, against the fp64 oracle's
matching definition on the same seeded inputs.  Sizes span several tiles and ragged tails."""
import math

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import il_oracle as orc
from paper_2010_04116_b200 import binding as il

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bf16(a: np.ndarray):
    """numpy fp64/fp32 -> (cuda bf16 tensor, its exact fp64 values)"""
    t = torch.tensor(a, dtype=torch.float32).to(torch.bfloat16).to(DEV)
    return t, t.float().cpu().numpy().astype(np.float64)


def _err_word():
    return torch.zeros(1, dtype=torch.int32, device=DEV)


def _rel(a, b):
    return np.linalg.norm(np.asarray(a, dtype=np.float64) - b) / max(np.linalg.norm(b), 1e-30)


GEMM_SHAPES = [(128, 256, 64), (300, 520, 200), (257, 136, 72), (4096, 2560, 256), (1000, 1024, 512)]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("layout", ["kk", "kmn", "mnmn"])
def test_gemm_layouts_fp32_out(M, N, K, layout):
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    A64 = rng.standard_normal((M, K))
    B64 = rng.standard_normal((N, K))
    a_mn = layout == "mnmn"
    b_mn = layout in ("kmn", "mnmn")
    # leading dimensions padded to a multiple of 8 elements, with garbage in the padding
    def store(mat64, mn):
        m = mat64.T if mn else mat64            # memory image [rows, cols]
        ld = (m.shape[1] + 7) // 8 * 8
        buf = rng.standard_normal((m.shape[0], ld))
        buf[:, :m.shape[1]] = m
        t, exact = _bf16(buf)
        e = exact[:, :m.shape[1]]
        return t, ld, (e.T if mn else e)
    At, lda, Ae = store(A64, a_mn)
    Bt, ldb, Be = store(B64, b_mn)
    ldc = (N + 3) // 4 * 4
    Ct = torch.full((M, ldc), 7.0, dtype=torch.float32, device=DEV)
    err = _err_word()
    il.op_gemm(M, N, K, At, lda, int(a_mn), Bt, ldb, int(b_mn), 4, err, C_=Ct, ldc=ldc)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = Ae @ Be.T
    got = Ct.cpu().numpy()
    assert _rel(got[:, :N], ref) < 2e-6
    if ldc > N:
        assert np.all(got[:, N:] == 7.0)       # nothing written outside the N valid columns
    # accumulate: C += A B^T
    il.op_gemm(M, N, K, At, lda, int(a_mn), Bt, ldb, int(b_mn), 4, err, C_=Ct, ldc=ldc, accumulate=1)
    torch.cuda.synchronize()
    assert _rel(Ct.cpu().numpy()[:, :N], 2 * ref) < 2e-6


def test_gemm_epilogues_forward():
    rng = np.random.default_rng(5)
    M, N, K = 384, 328, 136
    At, Ae = _bf16(rng.standard_normal((M, K)))
    Bt, Be = _bf16(rng.standard_normal((N, K)) * 0.2)
    bias = rng.standard_normal(N)
    bt = torch.tensor(bias, dtype=torch.float32, device=DEV)
    pre = Ae @ Be.T + bt.cpu().numpy().astype(np.float64)
    err = _err_word()
    # 0: bf16 out + bias
    C0 = torch.zeros((M, N), dtype=torch.bfloat16, device=DEV)
    il.op_gemm(M, N, K, At, K, 0, Bt, K, 0, 0, err, C_=C0, ldc=N, bias=bt)
    # 1: gelu'(pre) and gelu(pre)
    C1 = torch.zeros((M, N), dtype=torch.bfloat16, device=DEV)
    C2 = torch.zeros((M, N), dtype=torch.bfloat16, device=DEV)
    il.op_gemm(M, N, K, At, K, 0, Bt, K, 0, 1, err, C_=C1, ldc=N, C2=C2, bias=bt)
    # 2: fp32 residual, in place
    R = torch.tensor(rng.standard_normal((M, N)), dtype=torch.float32, device=DEV)
    R0 = R.cpu().numpy().astype(np.float64)
    il.op_gemm(M, N, K, At, K, 0, Bt, K, 0, 2, err, C_=R, ldc=N, bias=bt, resid=R)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert _rel(C0.float().cpu().numpy(), pre) < 3e-3
    assert _rel(C1.float().cpu().numpy(), orc.gelu_grad(pre)) < 3e-3
    assert _rel(C2.float().cpu().numpy(), orc.gelu(pre)) < 3e-3
    assert _rel(R.cpu().numpy(), R0 + pre) < 1e-6


def test_gemm_multiply_epilogue_with_stacked_rows():
    rng = np.random.default_rng(6)
    rows, s, N, K = 200, 2, 264, 128          # 2 stacked gradient streams share one saved gelu'
    M = rows * s
    At, Ae = _bf16(rng.standard_normal((M, K)))
    Wt, We = _bf16(rng.standard_normal((K, N)) * 0.3)      # dgrad: B stored [K, N] (MN-major)
    Ht, He = _bf16(rng.standard_normal((rows, N)))
    Ct = torch.zeros((M, N), dtype=torch.bfloat16, device=DEV)
    err = _err_word()
    cs = torch.zeros(N, dtype=torch.float32, device=DEV)
    il.op_gemm(M, N, K, At, K, 0, Wt, N, 1, 3, err, C_=Ct, ldc=N, aux=Ht, ld_aux=N, aux_rows=rows, colsum=cs)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = (Ae @ We) * np.tile(He, (s, 1))
    assert _rel(Ct.float().cpu().numpy(), ref) < 3e-3
    assert _rel(cs.cpu().numpy(), ref[:rows].sum(axis=0)) < 1e-5      # bias gradient from the first stream only


@pytest.mark.parametrize("V", [512, 1000, 50257])
def test_gemm_softmax_epilogues(V):
    """Online-softmax partials + dZ epilogue against full logits in fp64 (head of the auxiliary network)."""
    rng = np.random.default_rng(V)
    M, K = 200, 128
    Ut, Ue = _bf16(rng.standard_normal((M, K)))
    Wt, We = _bf16(rng.standard_normal((V, K)) * 0.3)
    tgt = rng.integers(0, V, size=M).astype(np.int32)
    tgt[0], tgt[1] = 0, V - 1
    tt = torch.tensor(tgt, device=DEV)
    ntiles = (V + 127) // 128
    pm = torch.zeros((M, ntiles), dtype=torch.float32, device=DEV)
    ps = torch.zeros((M, ntiles), dtype=torch.float32, device=DEV)
    tl = torch.zeros(M, dtype=torch.float32, device=DEV)
    err = _err_word()
    il.op_gemm(M, V, K, Ut, K, 0, Wt, K, 0, 5, err, targets=tt, part_max=pm, part_sum=ps, part_ld=ntiles, tgt_logit=tl)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    z = Ue @ We.T
    zmax = z.max(axis=1)
    lse_ref = zmax + np.log(np.exp(z - zmax[:, None]).sum(axis=1))
    pmn, psn = pm.cpu().numpy().astype(np.float64), ps.cpu().numpy().astype(np.float64)
    gmax = pmn.max(axis=1)
    lse = gmax + np.log((psn * np.exp(pmn - gmax[:, None])).sum(axis=1))
    assert np.max(np.abs(lse - lse_ref)) < 2e-5 * max(1.0, np.abs(lse_ref).max())
    assert np.max(np.abs(tl.cpu().numpy() - z[np.arange(M), tgt])) < 1e-4
    # the same call with C given also keeps the logits (bf16, padded row stride); statistics unchanged
    ldz = (V + 63) // 64 * 64
    zt = torch.full((M, ldz), 7.0, dtype=torch.bfloat16, device=DEV)
    pm2, ps2, tl2 = torch.zeros_like(pm), torch.zeros_like(ps), torch.zeros_like(tl)
    il.op_gemm(M, V, K, Ut, K, 0, Wt, K, 0, 5, err, C_=zt, ldc=ldz, targets=tt, part_max=pm2, part_sum=ps2,
               part_ld=ntiles, tgt_logit=tl2)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert torch.equal(pm2, pm) and torch.equal(ps2, ps) and torch.equal(tl2, tl)
    zg = zt.float().cpu().numpy()
    assert np.max(np.abs(zg[:, :V] - z)) <= 2.0 ** -8 * np.abs(z).max() + 1e-6     # one bf16 rounding
    assert np.all(zg[:, V:] == 7.0)
    # store_exp: what is kept is exp(logit), rounded once to bf16
    et = torch.full((M, ldz), 7.0, dtype=torch.bfloat16, device=DEV)
    il.op_gemm(M, V, K, Ut, K, 0, Wt, K, 0, 5, err, C_=et, ldc=ldz, targets=tt, part_max=pm2, part_sum=ps2,
               part_ld=ntiles, tgt_logit=tl2, store_exp=1)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    # with store_exp the partial sums are formed from the stored exponentials times one factor per 32-column
    # chunk: the same numbers up to rounding order
    assert torch.equal(pm2, pm) and torch.equal(tl2, tl)
    assert torch.allclose(ps2, ps, rtol=2e-6, atol=0)
    eg = et.float().cpu().numpy()
    assert np.max(np.abs(eg[:, :V] / np.exp(z) - 1.0)) < 2.0 ** -8 + 1e-5
    assert np.all(eg[:, V:] == 7.0)
    # dZ on a chunk that starts mid-vocabulary and runs past its end
    col0 = (V // 2) // 8 * 8
    nv = V - col0
    ldc = (nv + 7) // 8 * 8 + 8
    dz = torch.full((M, ldc), 3.0, dtype=torch.bfloat16, device=DEV)
    lse_t = torch.tensor(lse_ref, dtype=torch.float32, device=DEV)
    Wc = Wt[col0:]
    il.op_gemm(M, nv, K, Ut, K, 0, Wc, K, 0, 6, err, C_=dz, ldc=ldc, targets=tt, lse=lse_t, scale=1.0 / M, col0=col0)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    p = np.exp(z - lse_ref[:, None])
    p[np.arange(M), tgt] -= 1.0
    ref = (p / M)[:, col0:]
    got = dz.float().cpu().numpy()
    assert _rel(got[:, :nv], ref) < 4e-3
    assert np.all(got[:, nv:] == 3.0)


@pytest.mark.parametrize("B,T,H,dh", [(2, 64, 2, 32), (1, 200, 2, 64), (2, 256, 3, 64), (1, 192, 2, 80), (1, 130, 1, 128),
                                      (3, 128, 2, 256), (1, 300, 1, 256)])
def test_attention_forward_backward(B, T, H, dh):
    rng = np.random.default_rng(B * 1000 + T + dh)
    d = H * dh
    qkv_t, qkv = _bf16(rng.standard_normal((B * T, 3 * d)))
    o = torch.zeros((B * T, d), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros((B, H, T), dtype=torch.float32, device=DEV)
    il.op_attention_fwd(qkv_t, o, lse, B, T, H, dh)
    torch.cuda.synchronize()
    ref = orc.attention_fwd(qkv, B, T, H)
    assert _rel(o.float().cpu().numpy(), ref) < 6e-3
    # lse against the definition
    q = qkv[:, :d].reshape(B, T, H, dh).transpose(0, 2, 1, 3)
    k = qkv[:, d:2 * d].reshape(B, T, H, dh).transpose(0, 2, 1, 3)
    s = q @ k.transpose(0, 1, 3, 2) / math.sqrt(dh)
    s = np.where(np.triu(np.ones((T, T), dtype=bool), 1), -np.inf, s)
    smax = s.max(axis=-1)
    lse_ref = smax + np.log(np.exp(s - smax[..., None]).sum(axis=-1))
    assert np.max(np.abs(lse.cpu().numpy() - lse_ref)) < 2e-3
    # backward with two stacked gradient batches sharing the saved forward
    NB = 2 * B
    do_t, do = _bf16(rng.standard_normal((NB * T, d)))
    dqkv = torch.zeros((NB * T, 3 * d), dtype=torch.bfloat16, device=DEV)
    delta = torch.zeros(NB * H * T, dtype=torch.float32, device=DEV)
    il.op_attention_bwd(qkv_t, o, lse, do_t, dqkv, delta, NB, B, T, H, dh)
    torch.cuda.synchronize()
    got = dqkv.float().cpu().numpy()
    for j in range(2):
        refj = orc.attention_bwd(do[j * B * T:(j + 1) * B * T], qkv, B, T, H)
        gj = got[j * B * T:(j + 1) * B * T]
        for part, name in enumerate(["dq", "dk", "dv"]):
            sl = slice(part * d, (part + 1) * d)
            assert _rel(gj[:, sl], refj[:, sl]) < 1.5e-2, (j, name)


@pytest.mark.parametrize("B,T,H,dh,NB", [(2, 64, 2, 32, 2), (1, 200, 2, 64, 2), (2, 256, 3, 64, 4), (1, 1, 1, 64, 1),
                                         (1, 129, 2, 64, 1), (2, 1024, 2, 64, 2), (1, 700, 1, 32, 3)])
def test_attention_backward_one_sweep(B, T, H, dh, NB):
    """dK, dV and dQ from a single recomputation of the scores (dQ summed over key tiles in an fp32 accumulator):
    against the oracle, and against the two-kernel form (dK / dV take the same arithmetic path in both: equal bits)."""
    rng = np.random.default_rng(7 * B + T + dh + NB)
    d = H * dh
    qkv_t, qkv = _bf16(rng.standard_normal((B * T, 3 * d)))
    o = torch.zeros((B * T, d), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros((B, H, T), dtype=torch.float32, device=DEV)
    il.op_attention_fwd(qkv_t, o, lse, B, T, H, dh)
    do_t, do = _bf16(rng.standard_normal((NB * T, d)))
    two = torch.zeros((NB * T, 3 * d), dtype=torch.bfloat16, device=DEV)
    delta = torch.zeros(NB * H * T, dtype=torch.float32, device=DEV)
    il.op_attention_bwd(qkv_t, o, lse, do_t, two, delta, NB, B, T, H, dh)
    err = torch.zeros(1, dtype=torch.int32, device=DEV)
    for attempt in range(2):                      # twice: the accumulator holds the first call's values at the second
        one = torch.full((NB * T, 3 * d), 3.0, dtype=torch.bfloat16, device=DEV)
        acc = torch.full((NB * T, d), 5.0, dtype=torch.float32, device=DEV) if attempt == 0 else acc
        il.op_attention_bwd_one_sweep(qkv_t, o, lse, do_t, one, delta, acc, NB, B, T, H, dh, err_word=err)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        got = one.float().cpu().numpy()
        assert np.isfinite(got).all()
        for j in range(NB):
            refj = orc.attention_bwd(do[j * T:(j + 1) * T], qkv[(j % B) * T:(j % B + 1) * T], 1, T, H)
            gj = got[j * T:(j + 1) * T]
            for part, name in enumerate(["dq", "dk", "dv"]):
                sl = slice(part * d, (part + 1) * d)
                if np.linalg.norm(refj[:, sl]) < 1e-9:             # a single token: dQ and dK vanish identically
                    assert np.max(np.abs(gj[:, sl])) < 1e-5, (attempt, j, name)
                else:
                    assert _rel(gj[:, sl], refj[:, sl]) < 1.5e-2, (attempt, j, name)
        ref2 = two.float().cpu().numpy()
        assert np.array_equal(got[:, d:], ref2[:, d:])                 # dK, dV
        if T > 1:
            assert _rel(got[:, :d], ref2[:, :d]) < 4e-3                # dQ: the same values up to the order of the sum


@pytest.mark.parametrize("rows,d", [(64, 128), (1000, 768), (333, 2560)])
def test_layernorm_forward_backward(rows, d):
    rng = np.random.default_rng(rows + d)
    x = (rng.standard_normal((rows, d)) * 2 + 0.5).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(d)).astype(np.float32)
    b = (0.1 * rng.standard_normal(d)).astype(np.float32)
    xt, gt, bt = [torch.tensor(v, device=DEV) for v in (x, g, b)]
    y = torch.zeros((rows, d), dtype=torch.bfloat16, device=DEV)
    mean = torch.zeros(rows, dtype=torch.float32, device=DEV)
    rstd = torch.zeros(rows, dtype=torch.float32, device=DEV)
    il.op_layernorm_fwd(xt, gt, bt, y, mean, rstd, rows, d)
    torch.cuda.synchronize()
    yref, cache = orc.layernorm_fwd(x.astype(np.float64), g.astype(np.float64), b.astype(np.float64))
    assert _rel(y.float().cpu().numpy(), yref) < 3e-3
    assert np.allclose(mean.cpu().numpy(), x.astype(np.float64).mean(axis=1), atol=1e-5)
    assert np.allclose(rstd.cpu().numpy(), cache[1][:, 0], rtol=1e-5)
    # backward: two stacked streams, fp32 and bf16 dy, with residual
    s = 2
    for dy_f32 in (1, 0):
        dy64 = rng.standard_normal((s * rows, d))
        if dy_f32:
            dyt = torch.tensor(dy64, dtype=torch.float32, device=DEV)
            dye = dyt.cpu().numpy().astype(np.float64)
        else:
            dyt, dye = _bf16(dy64)
        res = torch.tensor(rng.standard_normal((s * rows, d)), dtype=torch.float32, device=DEV)
        res0 = res.cpu().numpy().astype(np.float64)
        dxb = torch.zeros((s * rows, d), dtype=torch.bfloat16, device=DEV)
        dg = torch.zeros(d, dtype=torch.float32, device=DEV)
        db = torch.zeros(d, dtype=torch.float32, device=DEV)
        il.op_layernorm_bwd(dyt, dy_f32, xt, mean, rstd, gt, res, res, dxb, dg, db, s * rows, rows, d)
        torch.cuda.synchronize()
        got = res.cpu().numpy()
        for j in range(s):
            dxr, dgr, dbr = orc.layernorm_bwd(dye[j * rows:(j + 1) * rows], cache, g.astype(np.float64))
            assert _rel(got[j * rows:(j + 1) * rows], res0[j * rows:(j + 1) * rows] + dxr) < 1e-5
            if j == 0:      # parameter gradients come from the first stream only
                assert _rel(dg.cpu().numpy(), dgr) < 1e-4
                assert _rel(db.cpu().numpy(), dbr) < 1e-4
        assert _rel(dxb.float().cpu().numpy(), got.astype(np.float64)) < 3e-3


@pytest.mark.parametrize("rows,d,s", [(40, 128, 1), (1000, 768, 2), (8192 + 13, 1024, 2), (300, 384, 3)])
def test_layernorm_backward_one_pass(rows, d, s):
    """The one-pass LayerNorm backward of the blocks: row part for s stacked streams, gamma / beta gradients and the
    column sums of its own output over the first stream, added to what the outputs already hold."""
    rng = np.random.default_rng(rows * 3 + d + s)
    x = (rng.standard_normal((rows, d)) * 2 + 0.5).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(d)).astype(np.float32)
    xt, gt = torch.tensor(x, device=DEV), torch.tensor(g, device=DEV)
    y = torch.zeros((rows, d), dtype=torch.bfloat16, device=DEV)
    mean = torch.zeros(rows, dtype=torch.float32, device=DEV)
    rstd = torch.zeros(rows, dtype=torch.float32, device=DEV)
    il.op_layernorm_fwd(xt, gt, torch.zeros(d, device=DEV), y, mean, rstd, rows, d)
    _, cache = orc.layernorm_fwd(x.astype(np.float64), g.astype(np.float64), np.zeros(d))
    dyt, dye = _bf16(rng.standard_normal((s * rows, d)))
    res = torch.tensor(rng.standard_normal((s * rows, d)), dtype=torch.float32, device=DEV)
    res0 = res.cpu().numpy().astype(np.float64)
    dxb = torch.zeros((s * rows, d), dtype=torch.bfloat16, device=DEV)
    start = [rng.standard_normal(d).astype(np.float32) for _ in range(3)]     # sums the outputs are added to
    dg, db, cs = [torch.tensor(v, device=DEV) for v in start]
    il.op_layernorm_bwd_fused(dyt, xt, mean, rstd, gt, res, res, dxb, dg, db, cs, s * rows, rows, d)   # dx aliases resid
    torch.cuda.synchronize()
    got = res.cpu().numpy().astype(np.float64)
    for j in range(s):
        dxr, dgr, dbr = orc.layernorm_bwd(dye[j * rows:(j + 1) * rows], cache, g.astype(np.float64))
        ref = res0[j * rows:(j + 1) * rows] + dxr
        assert _rel(got[j * rows:(j + 1) * rows], ref) < 1e-5
        if j == 0:
            assert _rel(dg.cpu().numpy() - start[0], dgr) < 1e-4
            assert _rel(db.cpu().numpy() - start[1], dbr) < 1e-4
            assert _rel(cs.cpu().numpy() - start[2], ref.sum(axis=0)) < 1e-4
    assert _rel(dxb.float().cpu().numpy(), got) < 3e-3
    with pytest.raises(il.ILError):          # widths outside its range are refused, not mishandled
        il.op_layernorm_bwd_fused(dyt, xt, mean, rstd, gt, res, res, dxb, dg, db, cs, s * rows, rows, 2560)


@pytest.mark.parametrize("split", [2, 4])
def test_gemm_split_k_adds_partial_sums(split):
    """wgrad layout with the contraction split over several work units per tile (atomic fp32 accumulation)."""
    rng = np.random.default_rng(split)
    M, N, K = 300, 264, 4096 + 72
    At, Ae = _bf16(rng.standard_normal((K, M + 4)))          # MN-major A: memory [K, M], ld padded
    Bt, Be = _bf16(rng.standard_normal((K, N)))
    Ct = torch.zeros((M, N), dtype=torch.float32, device=DEV)
    err = _err_word()
    il.op_gemm(M, N, K, At, M + 4, 1, Bt, N, 1, 4, err, C_=Ct, ldc=N, split_k=split)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = Ae[:, :M].T @ Be
    assert _rel(Ct.cpu().numpy(), ref) < 5e-6      # fp32 accumulation over K = 4168 plus the atomic partial sums


@pytest.mark.parametrize("M,N,K,layout,epi", [
    (512, 512, 128, (0, 0), 4),        # exactly one wide tile
    (1000, 700, 200, (0, 0), 0),       # ragged: the second wide tile has one and a bit column blocks
    (777, 1304, 136, (0, 1), 4),       # dgrad layout, three wide tiles, ragged rows
    (1304, 560, 264, (1, 1), 4),       # wgrad layout
    (640, 900, 320, (0, 0), 2),        # fp32 residual epilogue
    (600, 768, 192, (0, 1), 0),        # one and a half wide tiles: the last tile's second block is skipped whole
    (300, 1000, 128, (0, 0), 5),       # softmax partials: block index must follow the column, not the tile
])
def test_gemm_wide_tiles_match_square_tiles(M, N, K, layout, epi):
    """256 x 512 output tiles (two accumulators per tile, shared A slab) compute each element exactly as
    256 x 256 tiles do: same products, same order."""
    rng = np.random.default_rng(M + N + K)
    a_mn, b_mn = layout
    At, _ = _bf16(rng.standard_normal((K, M) if a_mn else (M, K)))
    Bt, _ = _bf16(rng.standard_normal((K, N) if b_mn else (N, K)) * 0.2)
    lda, ldb = (M if a_mn else K), (N if b_mn else K)
    ldc = (N + 7) // 8 * 8
    outs = []
    for tb in (1, 2):
        err = _err_word()
        kw = {}
        extra = []
        if epi == 0:
            Ct = torch.zeros((M, ldc), dtype=torch.bfloat16, device=DEV)
            kw["bias"] = torch.linspace(-1, 1, N, device=DEV)
        elif epi == 5:
            nt = (N + 127) // 128
            Ct = torch.zeros((M, ldc), dtype=torch.bfloat16, device=DEV)
            pm = torch.zeros((M, nt), device=DEV); ps = torch.zeros((M, nt), device=DEV); tl = torch.zeros(M, device=DEV)
            kw.update(targets=torch.tensor(rng.integers(0, N, size=M).astype(np.int32), device=DEV) if not outs else outs[0][1][3],
                      part_max=pm, part_sum=ps, part_ld=nt, tgt_logit=tl)
            extra = [pm, ps, tl, kw["targets"]]
        else:
            Ct = torch.zeros((M, ldc), dtype=torch.float32, device=DEV)
            if epi == 2:
                kw["resid"] = torch.full((M, ldc), 0.5, device=DEV)
        il.op_gemm(M, N, K, At, lda, a_mn, Bt, ldb, b_mn, epi, err, C_=Ct, ldc=ldc, tile_blocks=tb, **kw)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        outs.append((Ct.clone(), extra))
    assert torch.equal(outs[0][0], outs[1][0])
    for x, y in zip(outs[0][1], outs[1][1]):
        assert torch.equal(x, y)
    ref = (At.float().T if a_mn else At.float()) @ (Bt.float() if b_mn else Bt.float().T)
    got = outs[1][0][:, :N].float() - (0.5 if epi == 2 else 0.0) - (kw["bias"] if epi == 0 else 0.0)
    assert torch.linalg.norm(got - ref) / torch.linalg.norm(ref) < (4e-3 if epi in (0, 5) else 1e-5)


def test_gemm_row_scale_on_fp32_output():
    """Epilogue 4 with a per-row factor (the head's input gradient dU = diag(s) (E W)), with and without accumulation."""
    rng = np.random.default_rng(11)
    M, N, K = 300, 264, 520
    At, Ae = _bf16(rng.standard_normal((M, K)))
    Bt, Be = _bf16(rng.standard_normal((K, N)) * 0.3)          # MN-major B, as in dgrad
    sc = rng.uniform(0.1, 3.0, size=M)
    st = torch.tensor(sc, dtype=torch.float32, device=DEV)
    Ct = torch.full((M, N), 2.0, dtype=torch.float32, device=DEV)
    err = _err_word()
    il.op_gemm(M, N, K, At, K, 0, Bt, N, 1, 4, err, C_=Ct, ldc=N, rowscale=st)
    torch.cuda.synchronize()
    ref = (Ae @ Be) * st.cpu().numpy().astype(np.float64)[:, None]
    assert _rel(Ct.cpu().numpy(), ref) < 2e-6
    il.op_gemm(M, N, K, At, K, 0, Bt, N, 1, 4, err, C_=Ct, ldc=N, rowscale=st, accumulate=1)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert _rel(Ct.cpu().numpy(), 2 * ref) < 2e-6
