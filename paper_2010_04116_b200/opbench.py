"""Time one operator of the library at the GPT-2-medium-shaped sizes (8192 tokens, d 1024, 16 heads of 64, vocab 50257)
through the C ABI: useful for comparing kernel changes and as a small case for profiler captures.

    python -m paper_2010_04116_b200.opbench <op> [iterations] [gradient batches]

ops: logits (auxiliary head: vocabulary projection with the softmax / exp(logit) epilogue), plain (the same
contraction with a plain bf16 output), fc1 (first MLP projection with the GELU epilogue and its two outputs),
fc1_plain (the same contraction, bias and bf16 output only), dgelu (gradient through the second MLP projection,
multiplied by the saved GELU derivative, with the bias-gradient column sums; dgelu_nosum without them; dgelu_plain
the bare contraction), attn_fwd, attn_bwd (two kernels), attn_bwd_one (one sweep; gradient batches = stacked
gradient streams x 8).
"""
from __future__ import annotations

import sys

import torch

from . import binding as il

DEV = "cuda:0"
TILE = 0          # output tile width of the GEMMs: chosen by the library from the shape


def _timeit(name, fn, flops, iters, err):
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        fn()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / iters
    print(f"{name}: {ms * 1e3:.1f} us, {flops / ms / 1e9:.1f} TFLOP/s, device error word {int(err.item())}")


def main(argv):
    which = argv[1] if len(argv) > 1 else "logits"
    iters = int(argv[2]) if len(argv) > 2 else 10
    err = torch.zeros(1, dtype=torch.int32, device=DEV)
    if which in ("logits", "plain"):
        M, V, K = 8192, 50257, 1024
        ldz = (V + 63) // 64 * 64
        U = torch.randn(M, K, device=DEV).to(torch.bfloat16)
        W = (torch.randn(V, K, device=DEV) * 0.02).to(torch.bfloat16)
        E = torch.empty(M, ldz, dtype=torch.bfloat16, device=DEV)
        if which == "logits":
            tt = torch.randint(0, V, (M,), dtype=torch.int32, device=DEV)
            nt = (V + 127) // 128
            pm, ps = torch.zeros(M, nt, device=DEV), torch.zeros(M, nt, device=DEV)
            tl = torch.zeros(M, device=DEV)
            fn = lambda: il.op_gemm(M, V, K, U, K, 0, W, K, 0, 5, err, C_=E, ldc=ldz, targets=tt, part_max=pm,
                                    part_sum=ps, part_ld=nt, tgt_logit=tl, store_exp=1, tile_blocks=TILE)
        else:
            fn = lambda: il.op_gemm(M, V, K, U, K, 0, W, K, 0, 0, err, C_=E, ldc=ldz, tile_blocks=TILE)
        _timeit(which, fn, 2.0 * M * V * K, iters, err)
    elif which in ("fc1", "fc1_plain"):
        M, N, K = 8192, 4096, 1024
        X = torch.randn(M, K, device=DEV).to(torch.bfloat16)
        W = (torch.randn(N, K, device=DEV) * 0.02).to(torch.bfloat16)
        bias = torch.randn(N, device=DEV) * 0.02
        Y, Y2 = (torch.empty(M, N, dtype=torch.bfloat16, device=DEV) for _ in range(2))
        if which == "fc1":
            fn = lambda: il.op_gemm(M, N, K, X, K, 0, W, K, 0, 1, err, C_=Y, ldc=N, C2=Y2, bias=bias, tile_blocks=TILE)
        else:
            fn = lambda: il.op_gemm(M, N, K, X, K, 0, W, K, 0, 0, err, C_=Y, ldc=N, bias=bias, tile_blocks=TILE)
        _timeit(which, fn, 2.0 * M * N * K, iters, err)
    elif which in ("dgelu", "dgelu_nosum", "dgelu_plain"):
        R, N, K = 16384, 4096, 1024            # two stacked gradient streams of 8192 tokens
        dY = torch.randn(R, K, device=DEV).to(torch.bfloat16)
        W2 = (torch.randn(K, N, device=DEV) * 0.02).to(torch.bfloat16)      # [d, F]: read MN-major
        aux = torch.randn(R // 2, N, device=DEV).to(torch.bfloat16)
        out = torch.empty(R, N, dtype=torch.bfloat16, device=DEV)
        cs = torch.zeros(N, device=DEV)
        if which == "dgelu_plain":
            fn = lambda: il.op_gemm(R, N, K, dY, K, 0, W2, N, 1, 0, err, C_=out, ldc=N, tile_blocks=TILE or 1)
        else:
            fn = lambda: il.op_gemm(R, N, K, dY, K, 0, W2, N, 1, 3, err, C_=out, ldc=N, aux=aux, ld_aux=N,
                                    aux_rows=R // 2, colsum=cs if which == "dgelu" else None, tile_blocks=TILE)
        _timeit(which, fn, 2.0 * R * N * K, iters, err)
    elif which in ("attn_fwd", "attn_bwd", "attn_bwd_one"):
        B, T, H, dh = 8, 1024, 16, 64
        NB = int(argv[3]) if len(argv) > 3 else B
        d = H * dh
        qkv = torch.randn(B * T, 3 * d, device=DEV).to(torch.bfloat16)
        o = torch.empty(B * T, d, dtype=torch.bfloat16, device=DEV)
        lse = torch.empty(B * H * T, device=DEV)
        il.op_attention_fwd(qkv, o, lse, B, T, H, dh)
        causal = 2.0 * B * H * T * T * dh          # QK^T and PV over the lower triangle
        if which == "attn_fwd":
            _timeit(which, lambda: il.op_attention_fwd(qkv, o, lse, B, T, H, dh), causal, iters, err)
        else:
            do = torch.randn(NB * T, d, device=DEV).to(torch.bfloat16)
            dqkv = torch.empty(NB * T, 3 * d, dtype=torch.bfloat16, device=DEV)
            delta = torch.empty(NB * H * T, device=DEV)
            if which == "attn_bwd":
                fn = lambda: il.op_attention_bwd(qkv, o, lse, do, dqkv, delta, NB, B, T, H, dh)
            else:
                acc = torch.empty(NB * T, d, device=DEV)
                fn = lambda: il.op_attention_bwd_one_sweep(qkv, o, lse, do, dqkv, delta, acc, NB, B, T, H, dh, err_word=err)
            _timeit(which, fn, 2.5 * causal * NB / B, iters, err)
    else:
        raise SystemExit(__doc__)


if __name__ == "__main__":
    main(sys.argv)
