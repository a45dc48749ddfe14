"""Parity (GPU) of the paper-shaped extensions with the fp64 oracle, through the C ABI: auxiliary networks
that hold Transformer blocks (App. B.3) and mini-batches processed as micro-batches (Sec. 3.1).  Same
tolerances as the main parity tests: losses 1e-3 relative, gradients 2e-2 relative L2 per tensor."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import workloads as wl
from oracle import il_oracle as orc
from paper_2010_04116_b200 import ILError, Model

pytestmark = pytest.mark.gpu

LOSS_RTOL = 1e-3
GRAD_RTOL = 2e-2


def _compare(m, OG):
    for name in m.names:
        g = m.get_grad(name).astype(np.float64)
        ref = OG[name]
        den = np.linalg.norm(ref)
        if den == 0.0:
            assert np.all(g == 0.0), name
            continue
        rel = np.linalg.norm(g - ref) / den
        assert rel < GRAD_RTOL, (name, rel)


@pytest.mark.parametrize("rule,n,Lh", [("sum", 2, 2), ("mean", 2, 2), ("far", 3, 1), ("sum", 1, 1)])
def test_heads_with_transformer_blocks(rule, n, Lh):
    w = wl.Workload("auxblk", K=3, Lc=1, d=128, H=2, F=256, V=1000, T=96, B=2, n=n, zipf=True, Lh=Lh)
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, n, w.B, w.T, head_layers=Lh)
    try:
        assert m.names == [s[0] for s in wl.tensor_specs(w)]
        m.set_params(P)
        m.set_rule(rule)
        m.train_step(tok, tgt)
        losses = m.get_losses()
        m.sync()
        ol, OG = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n, rule=rule, head_layers=Lh)
        assert np.all(np.abs(losses - np.array(ol)) <= LOSS_RTOL * np.abs(np.array(ol))), (losses, ol)
        _compare(m, OG)
    finally:
        m.close()


@pytest.mark.parametrize("M,Lh,rule", [(2, 0, "sum"), (4, 1, "mean")])
def test_micro_batched_update_matches_the_whole_mini_batch(M, Lh, rule):
    """M micro-batch passes accumulate the gradient of the mini-batch: compared with the oracle's plain
    whole-batch step; then one AdamW update from the accumulated gradients."""
    w = wl.Workload("micro", K=3, Lc=1, d=128, H=2, F=256, V=1000, T=64, B=4, n=2, zipf=True, Lh=Lh)
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    per = w.B // M
    m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, per, w.T, head_layers=Lh)
    try:
        m.set_params(P)
        m.set_rule(rule)
        m.set_micro_batches(M)
        mean_losses = np.zeros(w.K)
        for mb in range(M):
            m.train_step(tok[mb * per:(mb + 1) * per], tgt[mb * per:(mb + 1) * per])
            mean_losses += m.get_losses() / M
            if mb + 1 < M:
                with pytest.raises(ILError):        # an update needs all M micro-batches
                    m.adamw_step(lr=1e-3)
        m.sync()
        ol, OG = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, 2, rule=rule, head_layers=Lh)
        assert np.all(np.abs(mean_losses - np.array(ol)) <= LOSS_RTOL * np.abs(np.array(ol))), (mean_losses, ol)
        _compare(m, OG)
        G = {name: m.get_grad(name).astype(np.float64) for name in m.names}
        hp = dict(lr=1e-3, beta1=0.9, beta2=0.98, eps=1e-9, weight_decay=0.0)     # weight decay 0: the paper's Adam
        m.adamw_step(**hp)
        m.sync()
        newP = orc.adamw_step(P, G, {}, 1, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], 0.0)
        for name in m.names:
            assert np.max(np.abs(m.get_param(name).astype(np.float64) - newP[name])) < 2e-6, name
        # the next update starts from overwritten gradients again
        m.train_minibatch(tok, tgt, M)
        m.sync()
        P2 = {name: m.get_param(name) for name in m.names}
        _, OG2 = orc.nwise_gradients(P2, tok, tgt, w.K, w.Lc, w.H, 2, rule=rule, head_layers=Lh)
        _compare(m, OG2)
        with pytest.raises(ILError):                # an update takes no more than M micro-batches
            m.train_step(tok[:per], tgt[:per])
    finally:
        m.close()


def test_paper_head_shape_dh256_short_sequences():
    """The paper's Transformer shape has 4 attention heads at d 1024, i.e. head dimension 256, on sequences of
    128 tokens (App. B.3): one module pair with 2-block auxiliary networks at those widths and a small vocabulary."""
    w = wl.Workload("dh256", K=2, Lc=1, d=1024, H=4, F=4096, V=1200, T=128, B=2, n=2, zipf=True, Lh=2)
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, w.B, w.T, head_layers=w.Lh)
    try:
        m.set_params(P)
        m.set_rule("mean")
        m.train_step(tok, tgt)
        losses = m.get_losses()
        m.sync()
        ol, OG = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, 2, rule="mean", head_layers=w.Lh)
        assert np.all(np.abs(losses - np.array(ol)) <= LOSS_RTOL * np.abs(np.array(ol))), (losses, ol)
        _compare(m, OG)
    finally:
        m.close()
