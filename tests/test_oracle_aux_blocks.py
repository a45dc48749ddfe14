"""Pins for the oracle's auxiliary networks with Transformer blocks (App. B.3: main network output ->
2 Transformer blocks -> embedding matrix) and for micro-batched steps (Sec. 3.1).  Each check compares
oracle/il_oracle.py with something other than itself: finite differences of the windowed loss sums
(forward passes only), torch autograd with detach() at the component boundaries, the parameter count
the paper prints, and the identity between a micro-batched step and the whole mini-batch."""
import numpy as np
import pytest
import torch
import torch.nn.functional as Fnn

import workloads as wl
from oracle import il_oracle as orc

TINY_H1 = wl.Workload("tiny-h1", K=3, Lc=1, d=8, H=2, F=16, V=11, T=5, B=2, n=2, zipf=False, Lh=1)
TINY_H2 = wl.Workload("tiny-h2", K=3, Lc=2, d=12, H=3, F=20, V=13, T=6, B=4, n=2, zipf=False, Lh=2)


def _setup(w, scale=8.0):
    P = {k: v.astype(np.float64) * scale for k, v in wl.draw_params(w).items()}
    for k in P:
        if k.endswith(".g"):
            P[k] = 1.0 + (P[k] / scale - 1.0) * scale
    tok, tgt = wl.draw_tokens(w)
    return P, tok, tgt


def test_module_parameter_count_matches_the_paper():
    # App. B.3: a module of 6 blocks (d 1024) with its auxiliary network has 152M parameters
    w = wl.CONFIGS["cfgP"]
    per_module = sum(int(np.prod(s)) for name, comp, _, s in wl.tensor_specs(w)
                     if comp == 1 and name not in ("wte", "wpe"))
    assert round(per_module / 1e6) == 152


def _window_sum(P, tok, tgt, w, k, n):
    L = orc.head_losses(P, tok, tgt, w.K, w.Lc, w.H, head_layers=w.Lh)
    return sum(L[h] for h in range(k, min(k + n - 1, w.K - 1) + 1))


@pytest.mark.parametrize("n", [1, 2, 3])
def test_finite_differences_with_head_blocks(n):
    w = TINY_H1
    P, tok, tgt = _setup(w)
    _, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n, head_layers=w.Lh)
    rng = np.random.default_rng(40 + n)
    h = 1e-5
    for name, comp, is_head, shape in wl.tensor_specs(w):
        size = int(np.prod(shape))
        for _ in range(2):
            flat = int(rng.integers(0, size))
            idx = np.unravel_index(flat, shape)
            if name == "wte":
                idx = (int(tok.reshape(-1)[flat % tok.size]), idx[1])
            if is_head:   # head parameters (its blocks included) see their own loss only
                fn = lambda: orc.head_losses(P, tok, tgt, w.K, w.Lc, w.H, head_layers=w.Lh)[comp]
            else:
                fn = lambda: _window_sum(P, tok, tgt, w, comp, n)
            old = P[name][idx]
            P[name][idx] = old + h
            fp = fn()
            P[name][idx] = old - h
            fm = fn()
            P[name][idx] = old
            fd = (fp - fm) / (2 * h)
            g = G[name][idx]
            # central differences carry ~1e-10 of absolute truncation and rounding noise at this step
            assert abs(fd - g) < 1e-6 * max(abs(fd), abs(g)) + 1e-9, (name, idx, fd, g)


def _torch_blocks(Pt, x, prefixes, w):
    B, T, H, d = w.B, w.T, w.H, w.d
    dh = d // H
    for p in prefixes:
        y = Fnn.layer_norm(x, (d,), Pt[p + "ln1.g"], Pt[p + "ln1.b"], eps=1e-5)
        qkv = Fnn.linear(y, Pt[p + "attn.wqkv"], Pt[p + "attn.bqkv"])
        q, kk, v = [z.reshape(B, T, H, dh).permute(0, 2, 1, 3) for z in qkv.split(d, dim=1)]
        o = Fnn.scaled_dot_product_attention(q, kk, v, is_causal=True).permute(0, 2, 1, 3).reshape(B * T, d)
        x = x + Fnn.linear(o, Pt[p + "attn.wo"], Pt[p + "attn.bo"])
        y = Fnn.layer_norm(x, (d,), Pt[p + "ln2.g"], Pt[p + "ln2.b"], eps=1e-5)
        hh = Fnn.gelu(Fnn.linear(y, Pt[p + "mlp.w1"], Pt[p + "mlp.b1"]), approximate="tanh")
        x = x + Fnn.linear(hh, Pt[p + "mlp.w2"], Pt[p + "mlp.b2"])
    return x


def _torch_nwise(P, tok, tgt, w, n):
    Pt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in P.items()}
    tt = torch.tensor(tok.reshape(-1), dtype=torch.long)
    yy = torch.tensor(tgt.reshape(-1), dtype=torch.long)
    pos = torch.arange(w.T).repeat(w.B)
    comp = lambda k: [f"c{k}.l{l}." for l in range(w.Lc)]
    a = [Pt["wte"][tt] + Pt["wpe"][pos]]
    for k in range(w.K):
        a.append(_torch_blocks(Pt, a[-1], comp(k), w))
    total, losses = 0.0, []
    for h in range(w.K):
        start = max(h + 1 - n, 0)
        x = a[start] if start == 0 else a[start].detach()
        for k in range(start, h + 1):
            x = _torch_blocks(Pt, x, comp(k), w)
        x = _torch_blocks(Pt, x, [f"head{h}.l{j}." for j in range(w.Lh)], w)
        u = Fnn.layer_norm(x, (w.d,), Pt[f"head{h}.ln.g"], Pt[f"head{h}.ln.b"], eps=1e-5)
        L = Fnn.cross_entropy(Fnn.linear(u, Pt[f"head{h}.w"]), yy)
        losses.append(L.item())
        total = total + L
    total.backward()
    return losses, {k: (v.grad.numpy() if v.grad is not None else np.zeros(v.shape)) for k, v in Pt.items()}


@pytest.mark.parametrize("w,n", [(TINY_H1, 1), (TINY_H1, 3), (TINY_H2, 2)])
def test_head_blocks_match_autograd_with_detach(w, n):
    P, tok, tgt = _setup(w)
    losses, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n, head_layers=w.Lh)
    tl, TG = _torch_nwise(P, tok, tgt, w, n)
    assert np.allclose(losses, tl, rtol=1e-12)
    for name in P:
        den = max(np.linalg.norm(TG[name]), 1e-30)
        assert np.linalg.norm(G[name] - TG[name]) / den < 1e-10, name


def test_head_blocks_of_other_heads_do_not_matter_to_a_head():
    # parameters inside head 0's blocks change head 0's loss and no other
    w = TINY_H1
    P, tok, tgt = _setup(w)
    L0 = orc.head_losses(P, tok, tgt, w.K, w.Lc, w.H, head_layers=w.Lh)
    P["head0.l0.mlp.w2"] = P["head0.l0.mlp.w2"] * 1.5
    L1 = orc.head_losses(P, tok, tgt, w.K, w.Lc, w.H, head_layers=w.Lh)
    assert L0[0] != L1[0] and L0[1:] == L1[1:]


@pytest.mark.parametrize("M", [2, 4])
@pytest.mark.parametrize("rule", ["sum", "mean"])
def test_micro_batched_step_equals_the_whole_mini_batch(M, rule):
    # equal-sized micro-batches: the mean of their mean-loss gradients is the mini-batch's (Sec. 3.1)
    w = TINY_H2
    P, tok, tgt = _setup(w)
    l1, G1 = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, 2, rule=rule, head_layers=w.Lh)
    lm, Gm = orc.nwise_gradients_microbatched(P, tok, tgt, w.K, w.Lc, w.H, 2, M, rule=rule, head_layers=w.Lh)
    assert np.allclose(l1, lm, rtol=1e-12)
    for name in P:
        den = max(np.linalg.norm(G1[name]), 1e-30)
        assert np.linalg.norm(G1[name] - Gm[name]) / den < 1e-11, name
    with pytest.raises(ValueError):
        orc.nwise_gradients_microbatched(P, tok, tgt, w.K, w.Lc, w.H, 2, 3)
