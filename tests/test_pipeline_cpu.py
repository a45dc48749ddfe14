"""The pipeline placement's exchange schedule on CPU, two gloo ranks (no GPU).

The paper places one module per accelerator; activations go to the next accelerator, gradients to the previous one
(Sec. 3, Fig. 3), and under the n-wise rule a head's gradient crosses at most n-1 boundaries.  The library states
which tensors cross which boundary in il_pipeline_transfers.  Here two processes each own half of the components
of a tiny network, compute their components with the fp64 oracle's block functions, and exchange over gloo exactly
the tensors that plan lists, in its order, and nothing else.  If the plan were missing a tensor, carried one too
far, or ordered the two sides differently, the gradients would differ from the oracle's single-process n-wise
gradients (or the ranks would dead-lock against the test's timeout)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

K, LC, D, H, F, V, T, B = 4, 1, 8, 2, 16, 11, 5, 2


def _owner(k):
    return 0 if k < K // 2 else 1


def _run_rank(rank, n, rule):
    import workloads as wl
    from oracle import il_oracle as orc
    import paper_2010_04116_b200 as pkg

    w = wl.Workload("pipe", K=K, Lc=LC, d=D, H=H, F=F, V=V, T=T, B=B, n=n, zipf=False)
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    plan = pkg.pipeline_transfers(K, n, rule)
    fwd = [r for r in plan if r[0] == 0]
    back = {b: [r[2] for r in plan if r[0] == 1 and r[1] == b] for b in range(K - 1)}
    sent = 0

    def send(x, to):
        nonlocal sent
        sent += 1
        dist.send(torch.from_numpy(np.ascontiguousarray(x)), dst=to)

    def recv(frm):
        t = torch.empty(B * T, D, dtype=torch.float64)
        dist.recv(t, src=frm)
        return t.numpy().copy()

    # ---- forward: a_{b+1} crosses boundary b
    a, caches = {}, {}
    if rank == _owner(0):
        a[0] = orc.embed_fwd(tok, P)
    for k in range(K):
        if _owner(k) == rank:
            a[k + 1], caches[k] = orc.component_fwd(a[k], P, k, LC, B, T, H)
        if k < K - 1:
            assert (0, k, -1) in fwd
            if _owner(k) == rank and _owner(k + 1) != rank:
                send(a[k + 1], _owner(k + 1))
            elif _owner(k + 1) == rank and _owner(k) != rank:
                a[k + 1] = recv(_owner(k))

    # ---- heads and backward, components from the top down
    G, losses, out = {}, {}, {}
    for k in reversed(range(K)):
        if _owner(k) != rank:
            continue
        loss, ghead, hg = orc.head_loss(a[k + 1], tgt, P, k, True)
        losses[k] = loss
        G.update(hg)
        incoming = {}
        if k < K - 1:
            for ident in back[k]:
                incoming[ident] = out[k + 1][ident] if _owner(k + 1) == rank else recv(_owner(k + 1))
        out[k] = {}
        below = back[k - 1] if k > 0 else []
        if rule == "sum":
            terms = pkg.nwise_streams(K, n, k)
            assert set(incoming) <= set(terms)
            U = {t: ghead + incoming.get(t, 0.0) for t in terms}
            dx_first = orc.component_bwd(U[terms[0]], caches[k], P, k, B, T, H, G)      # all heads: parameter gradients
            for t in below:
                out[k][t] = dx_first if t == terms[0] else orc.component_bwd(U[t], caches[k], P, k, B, T, H, {})
            if k == 0:
                orc.embed_bwd(dx_first, tok, P, G)
        else:
            hi = min(k + n - 1, K - 1)
            g = {k: ghead}
            g.update(incoming)
            comb = 0.0
            for h in range(k, hi + 1):
                wgt = orc.head_weight(k, h, n, K, rule)
                if wgt != 0.0:
                    comb = comb + wgt * g[h]          # KeyError here = the plan did not deliver a head it needs
            dx_comb = orc.component_bwd(comb, caches[k], P, k, B, T, H, G)
            for h in below:
                out[k][h] = orc.component_bwd(g[h], caches[k], P, k, B, T, H, {})
            if k == 0:
                orc.embed_bwd(dx_comb, tok, P, G)
        if k > 0 and _owner(k - 1) != rank:
            for ident in below:
                send(out[k][ident], _owner(k - 1))

    # ---- compare what this rank owns with the oracle's single-process step
    ol, OG = orc.nwise_gradients(P, tok, tgt, K, LC, H, n, rule=rule)
    for k, l in losses.items():
        assert abs(l - ol[k]) < 1e-12
    mine = [nm for nm, comp, _, _ in wl.tensor_specs(w) if _owner(comp) == rank]
    for nm in mine:
        ref = OG[nm]
        got = G.get(nm, np.zeros_like(ref))
        assert np.allclose(got, ref, rtol=1e-9, atol=1e-13), (rank, nm)
    # rank 1 sends across the one cross-rank boundary: one activation forward never (it receives it), and at most
    # n-1 gradients back; rank 0 sends the activation only
    cross = K // 2 - 1
    expect = 1 if rank == 0 else len(back[cross])
    assert sent == expect, (rank, sent, expect)
    assert len(back[cross]) <= n - 1


def _worker(rank, world, port, n, rule):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        _run_rank(rank, n, rule)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
@pytest.mark.parametrize("rule,port0", [("sum", 29700), ("far", 29710), ("mean", 29720)])
def test_two_ranks_exchange_exactly_the_planned_tensors(rule, port0):
    for n in range(1, K + 1):
        mp.spawn(_worker, args=(2, port0 + n, n, rule), nprocs=2, join=True)
