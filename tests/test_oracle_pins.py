"""Pins for the fp64 oracle: everything here checks oracle/il_oracle.py against something
other than itself — brute-force loops, closed forms, finite differences of an independent
formula (the windowed loss sum), torch's autograd with explicit detach() at component
boundaries, and the structural invariants of the n-wise rule (Sec. 3, Fig. 2)."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as Fnn

import workloads as wl
from oracle import il_oracle as orc

TINY = wl.Workload("tiny", K=3, Lc=1, d=8, H=2, F=16, V=11, T=5, B=2, n=2, zipf=False)
TINY2 = wl.Workload("tiny2", K=4, Lc=2, d=12, H=3, F=20, V=13, T=6, B=2, n=2, zipf=False)


def _setup(w, scale=8.0):
    # larger-than-init weights so that every non-linearity is exercised away from its linear regime
    P = {k: (v.astype(np.float64) * (1.0 if k.endswith(".g") else scale)) for k, v in wl.draw_params(w).items()}
    for k in P:
        if k.endswith(".g"):
            P[k] = 1.0 + (P[k] - 1.0) * scale
    tok, tgt = wl.draw_tokens(w)
    return P, tok, tgt


# ------------------------------------------------------------------ elementary pieces

def test_gelu_matches_library_and_fd():
    x = np.linspace(-4, 4, 101)
    ref = Fnn.gelu(torch.tensor(x), approximate="tanh").numpy()
    assert np.allclose(orc.gelu(x), ref, atol=1e-14)
    h = 1e-6
    fd = (orc.gelu(x + h) - orc.gelu(x - h)) / (2 * h)
    assert np.allclose(orc.gelu_grad(x), fd, atol=1e-8)
    # hand value: gelu(1) = 0.5 (1 + tanh(sqrt(2/pi) * 1.044715))
    assert abs(orc.gelu(np.array([1.0]))[0] - 0.5 * (1 + math.tanh(math.sqrt(2 / math.pi) * 1.044715))) < 1e-15


def test_layernorm_matches_library():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((7, 10)) * 3 + 1
    g = rng.standard_normal(10)
    b = rng.standard_normal(10)
    y, cache = orc.layernorm_fwd(x, g, b)
    xt = torch.tensor(x, requires_grad=True)
    gt = torch.tensor(g, requires_grad=True)
    bt = torch.tensor(b, requires_grad=True)
    yt = Fnn.layer_norm(xt, (10,), gt, bt, eps=1e-5)
    assert np.allclose(y, yt.detach().numpy(), atol=1e-13)
    dy = rng.standard_normal((7, 10))
    yt.backward(torch.tensor(dy))
    dx, dg, db = orc.layernorm_bwd(dy, cache, g)
    assert np.allclose(dx, xt.grad.numpy(), atol=1e-12)
    assert np.allclose(dg, gt.grad.numpy(), atol=1e-12)
    assert np.allclose(db, bt.grad.numpy(), atol=1e-12)
    # rows of a normalised output (g=1, b=0) have mean 0 and variance var/(var+eps)
    y0, _ = orc.layernorm_fwd(x, np.ones(10), np.zeros(10))
    assert np.allclose(y0.mean(axis=1), 0, atol=1e-14)


def _attention_loops(qkv, B, T, H):
    """Causal attention written with python loops over every (batch, head, query)."""
    d = qkv.shape[1] // 3
    dh = d // H
    out = np.zeros((B * T, d))
    for b in range(B):
        for h in range(H):
            for i in range(T):
                q = qkv[b * T + i, h * dh:(h + 1) * dh]
                sc = []
                for j in range(i + 1):
                    kk = qkv[b * T + j, d + h * dh: d + (h + 1) * dh]
                    sc.append(sum(q[e] * kk[e] for e in range(dh)) / math.sqrt(dh))
                m = max(sc)
                ex = [math.exp(s - m) for s in sc]
                Z = sum(ex)
                for j in range(i + 1):
                    v = qkv[b * T + j, 2 * d + h * dh: 2 * d + (h + 1) * dh]
                    out[b * T + i, h * dh:(h + 1) * dh] += ex[j] / Z * v
    return out


def test_attention_brute_force_and_library():
    rng = np.random.default_rng(1)
    B, T, H, dh = 2, 5, 3, 4
    d = H * dh
    qkv = rng.standard_normal((B * T, 3 * d))
    o = orc.attention_fwd(qkv, B, T, H)
    assert np.allclose(o, _attention_loops(qkv, B, T, H), atol=1e-13)
    # library routine + autograd for the backward
    t = torch.tensor(qkv, requires_grad=True)
    q, k, v = [z.reshape(B, T, H, dh).permute(0, 2, 1, 3) for z in t.split(d, dim=1)]
    ot = Fnn.scaled_dot_product_attention(q, k, v, is_causal=True).permute(0, 2, 1, 3).reshape(B * T, d)
    assert np.allclose(o, ot.detach().numpy(), atol=1e-12)
    do = rng.standard_normal((B * T, d))
    ot.backward(torch.tensor(do))
    assert np.allclose(orc.attention_bwd(do, qkv, B, T, H), t.grad.numpy(), atol=1e-12)


def test_first_position_attends_only_to_itself():
    rng = np.random.default_rng(2)
    B, T, H, dh = 1, 4, 2, 4
    d = H * dh
    qkv = rng.standard_normal((B * T, 3 * d))
    o = orc.attention_fwd(qkv, B, T, H)
    assert np.allclose(o[0], qkv[0, 2 * d:], atol=1e-14)


def _head_loops(a, tgt, g, b, W):
    N, d = a.shape
    V = W.shape[0]
    tot = 0.0
    for i in range(N):
        mu = sum(a[i]) / d
        var = sum((a[i] - mu) ** 2) / d
        u = [(a[i, e] - mu) / math.sqrt(var + 1e-5) * g[e] + b[e] for e in range(d)]
        z = [sum(u[e] * W[v, e] for e in range(d)) for v in range(V)]
        m = max(z)
        lse = m + math.log(sum(math.exp(zz - m) for zz in z))
        tot += lse - z[tgt[i]]
    return tot / N


def test_head_loss_brute_force_and_lnV():
    rng = np.random.default_rng(3)
    N, d, V = 6, 5, 9
    a = rng.standard_normal((N, d))
    tgt = rng.integers(0, V, size=N)
    P = {"head0.ln.g": rng.standard_normal(d), "head0.ln.b": rng.standard_normal(d),
         "head0.w": rng.standard_normal((V, d))}
    loss, _, _ = orc.head_loss(a, tgt, P, 0, False, row_block=4)
    assert abs(loss - _head_loops(a, tgt, P["head0.ln.g"], P["head0.ln.b"], P["head0.w"])) < 1e-13
    ref = Fnn.cross_entropy(torch.tensor(orc.layernorm_fwd(a, P["head0.ln.g"], P["head0.ln.b"])[0] @ P["head0.w"].T),
                            torch.tensor(tgt)).item()
    assert abs(loss - ref) < 1e-13
    # a head whose projection is all zeros predicts the uniform distribution: loss = ln V
    P["head0.w"] = np.zeros((V, d))
    loss0, da, hg = orc.head_loss(a, tgt, P, 0, True)
    assert abs(loss0 - math.log(V)) < 1e-14
    assert np.allclose(da, 0)                       # nothing flows back through a zero projection
    # rows of dz sum to zero => column sums of dW weighted by ... ; simplest consequence: sum_v dW[v,:] = 0
    assert np.allclose(hg["head0.w"].sum(axis=0), 0, atol=1e-14)


def test_causal_mask_future_tokens_do_not_change_past_losses():
    w = TINY
    P, tok, tgt = _setup(w)
    a, _ = orc.forward_all(P, tok, w.K, w.Lc, w.H)
    tok2 = tok.copy()
    t_change = 3
    tok2[:, t_change] = (tok2[:, t_change] + 1) % w.V
    a2, _ = orc.forward_all(P, tok2, w.K, w.Lc, w.H)
    for k in range(w.K + 1):
        x = a[k].reshape(w.B, w.T, -1)
        x2 = a2[k].reshape(w.B, w.T, -1)
        assert np.array_equal(x[:, :t_change], x2[:, :t_change])
        assert not np.allclose(x[:, t_change:], x2[:, t_change:])


# ------------------------------------------------------------------ the n-wise rule

def _window_sum(P, tok, tgt, w, k, n):
    """Independent formula: sum of the losses of the heads whose window covers component k."""
    L = orc.head_losses(P, tok, tgt, w.K, w.Lc, w.H)
    return sum(L[h] for h in range(k, min(k + n - 1, w.K - 1) + 1))


def _fd(P, name, idx, fn, h=1e-5):
    old = P[name][idx]
    P[name][idx] = old + h
    fp = fn()
    P[name][idx] = old - h
    fm = fn()
    P[name][idx] = old
    return (fp - fm) / (2 * h)


@pytest.mark.parametrize("n", [1, 2, 3])
def test_finite_differences_of_windowed_loss_sums(n):
    w = TINY
    P, tok, tgt = _setup(w)
    losses, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n)
    rng = np.random.default_rng(10 + n)
    specs = wl.tensor_specs(w)
    worst = 0.0
    for name, comp, is_head, shape in specs:
        size = int(np.prod(shape))
        for _ in range(3):
            flat = int(rng.integers(0, size))
            idx = np.unravel_index(flat, shape)
            if name == "wte":  # pick a row that occurs in the batch
                idx = (int(tok.reshape(-1)[flat % tok.size]), idx[1])
            if is_head:
                fn = lambda: orc.head_losses(P, tok, tgt, w.K, w.Lc, w.H)[comp]
            else:
                fn = lambda: _window_sum(P, tok, tgt, w, comp, n)
            fd = _fd(P, name, idx, fn)
            g = G[name][idx]
            err = abs(fd - g) / max(abs(fd), abs(g), 1e-7)
            worst = max(worst, err)
            assert err < 1e-6, (name, idx, fd, g)
    assert worst < 1e-6


def _torch_forward_from(Pt, x, k0, k1, w):
    """components k0..k1-1 applied to x with torch library ops (independent of the oracle's code)."""
    B, T, H, d = w.B, w.T, w.H, w.d
    dh = d // H
    for k in range(k0, k1):
        for l in range(w.Lc):
            p = f"c{k}.l{l}."
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
    """n-wise gradients by autograd: for each head, detach the activation n boundaries below it."""
    Pt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in P.items()}
    tt = torch.tensor(tok.reshape(-1), dtype=torch.long)
    yy = torch.tensor(tgt.reshape(-1), dtype=torch.long)
    pos = torch.arange(w.T).repeat(w.B)
    a = [Pt["wte"][tt] + Pt["wpe"][pos]]
    for k in range(w.K):
        a.append(_torch_forward_from(Pt, a[-1], k, k + 1, w))
    total = 0.0
    losses = []
    for h in range(w.K):
        start = max(h + 1 - n, 0)                    # index into a[]: the stopped boundary
        x = a[start] if start == 0 else a[start].detach()
        x = _torch_forward_from(Pt, x, start, h + 1, w)
        u = Fnn.layer_norm(x, (w.d,), Pt[f"head{h}.ln.g"], Pt[f"head{h}.ln.b"], eps=1e-5)
        L = Fnn.cross_entropy(Fnn.linear(u, Pt[f"head{h}.w"]), yy)
        losses.append(L.item())
        total = total + L
    total.backward()
    return losses, {k: (v.grad.numpy() if v.grad is not None else np.zeros(v.shape)) for k, v in Pt.items()}


@pytest.mark.parametrize("w,n", [(TINY, 1), (TINY, 2), (TINY, 3), (TINY2, 1), (TINY2, 2), (TINY2, 3), (TINY2, 4)])
def test_matches_autograd_with_detach_at_boundaries(w, n):
    P, tok, tgt = _setup(w)
    losses, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n)
    tl, TG = _torch_nwise(P, tok, tgt, w, n)
    assert np.allclose(losses, tl, rtol=1e-12)
    for name in P:
        den = max(np.linalg.norm(TG[name]), 1e-30)
        assert np.linalg.norm(G[name] - TG[name]) / den < 1e-10, name


def test_n_equals_K_is_full_backprop_of_summed_losses():
    w = TINY2
    P, tok, tgt = _setup(w)
    _, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, w.K)
    # plain autograd of sum_k L_k, nothing detached
    Pt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in P.items()}
    tt = torch.tensor(tok.reshape(-1), dtype=torch.long)
    yy = torch.tensor(tgt.reshape(-1), dtype=torch.long)
    x = Pt["wte"][tt] + Pt["wpe"][torch.arange(w.T).repeat(w.B)]
    total = 0.0
    for k in range(w.K):
        x = _torch_forward_from(Pt, x, k, k + 1, w)
        u = Fnn.layer_norm(x, (w.d,), Pt[f"head{k}.ln.g"], Pt[f"head{k}.ln.b"], eps=1e-5)
        total = total + Fnn.cross_entropy(Fnn.linear(u, Pt[f"head{k}.w"]), yy)
    total.backward()
    for name in P:
        assert np.allclose(G[name], Pt[name].grad.numpy(), rtol=1e-9, atol=1e-13), name


def test_one_wise_is_local():
    """n=1: component k and head k see only L_k (Sec. 3, local training)."""
    w = TINY
    P, tok, tgt = _setup(w)
    _, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, 1)
    P2 = {k: v.copy() for k, v in P.items()}
    rng = np.random.default_rng(5)
    P2["head2.w"] = rng.standard_normal(P["head2.w"].shape)     # disturb a higher head
    P2["head2.ln.g"] = rng.standard_normal(P["head2.ln.g"].shape)
    _, G2 = orc.nwise_gradients(P2, tok, tgt, w.K, w.Lc, w.H, 1)
    for name, comp, is_head, _ in wl.tensor_specs(w):
        if comp < 2:
            assert np.array_equal(G[name], G2[name]), name
    # and with n=2 component 1 does see head 2, component 0 still does not
    _, H1 = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, 2)
    _, H2 = orc.nwise_gradients(P2, tok, tgt, w.K, w.Lc, w.H, 2)
    assert not np.allclose(H1["c1.l0.mlp.w1"], H2["c1.l0.mlp.w1"])
    assert np.array_equal(H1["c0.l0.mlp.w1"], H2["c0.l0.mlp.w1"])
    assert np.array_equal(H1["wte"], H2["wte"])


def test_nesting_and_saturation():
    """G_n - G_{n-1} on component k is the plain gradient of L_{k+n-1}; head grads do not depend on n;
    component k's gradient stops changing once its window reaches the top head."""
    w = TINY2
    P, tok, tgt = _setup(w)
    Gs = {n: orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n)[1] for n in range(1, w.K + 1)}
    specs = wl.tensor_specs(w)
    for n in range(2, w.K + 1):
        for name, comp, is_head, _ in specs:
            if is_head:
                assert np.array_equal(Gs[n][name], Gs[1][name])
                continue
            h = comp + n - 1
            diff = Gs[n][name] - Gs[n - 1][name]
            if h > w.K - 1:
                assert np.array_equal(diff, np.zeros_like(diff)), (n, name)
            else:
                only = [0.0] * w.K
                only[h] = 1.0
                _, Gh = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, w.K, head_weights=only)
                assert np.allclose(diff, Gh[name], rtol=1e-9, atol=1e-14), (n, name)


def test_single_component_is_plain_training():
    w = wl.Workload("k1", K=1, Lc=2, d=8, H=2, F=16, V=11, T=5, B=2, n=1, zipf=False)
    P, tok, tgt = _setup(w)
    losses, G = orc.nwise_gradients(P, tok, tgt, 1, w.Lc, w.H, 1)
    tl, TG = _torch_nwise(P, tok, tgt, w, 1)
    assert np.allclose(losses, tl)
    for name in P:
        assert np.allclose(G[name], TG[name], rtol=1e-9, atol=1e-13)
    with pytest.raises(ValueError):
        orc.nwise_gradients(P, tok, tgt, 1, w.Lc, w.H, 2)


def test_embedding_gradient_counts_repeated_tokens():
    w = wl.Workload("emb", K=1, Lc=1, d=8, H=2, F=16, V=3, T=6, B=2, n=1, zipf=False)
    P, tok, tgt = _setup(w)
    G = {}
    dx = np.ones((w.B * w.T, w.d))
    orc.embed_bwd(dx, tok, P, G)
    counts = np.bincount(tok.reshape(-1), minlength=w.V)
    assert np.array_equal(G["wte"][:, 0], counts.astype(float))
    assert np.array_equal(G["wpe"][:, 0], np.full(w.T, w.B, dtype=float))


# ------------------------------------------------------------------ optimiser

def test_adamw_first_step_closed_form():
    rng = np.random.default_rng(7)
    P = {"w": rng.standard_normal((4, 3)), "b": rng.standard_normal(3)}
    G = {"w": rng.standard_normal((4, 3)), "b": rng.standard_normal(3)}
    st = {}
    lr, eps, wd = 1e-2, 1e-9, 0.1
    out = orc.adamw_step(P, G, st, 1, lr, 0.9, 0.98, eps, wd)
    # from zero state mhat = g, vhat = g^2: p - lr (g/(|g|+eps) + wd p); decay on matrices only
    assert np.allclose(out["w"], P["w"] - lr * (G["w"] / (np.abs(G["w"]) + eps) + wd * P["w"]), atol=1e-15)
    assert np.allclose(out["b"], P["b"] - lr * (G["b"] / (np.abs(G["b"]) + eps)), atol=1e-15)
    # constant gradient: mhat stays g, vhat stays g^2 at every step => same step size every time
    p = P
    for t in range(2, 6):
        new = orc.adamw_step(p, G, st, t, lr, 0.9, 0.98, eps, 0.0)
        assert np.allclose(new["b"] - p["b"], -lr * np.sign(G["b"]), atol=1e-9)
        p = new


def test_adamw_matches_library():
    rng = np.random.default_rng(8)
    p0 = rng.standard_normal((5, 4))
    pt = torch.tensor(p0.copy(), requires_grad=True)
    opt = torch.optim.AdamW([pt], lr=3e-3, betas=(0.9, 0.98), eps=1e-9, weight_decay=0.05)
    P = {"w": p0.copy()}
    st = {}
    for t in range(1, 5):
        g = rng.standard_normal((5, 4))
        pt.grad = torch.tensor(g)
        opt.step()
        P = orc.adamw_step(P, {"w": g}, st, t, 3e-3, 0.9, 0.98, 1e-9, 0.05)
        assert np.allclose(P["w"], pt.detach().numpy(), rtol=1e-10, atol=1e-12)


def test_lr_schedule_peak_at_warmup():
    # App. B.3: d^-0.5 min(step^-0.5, step warmup^-1.5); both branches meet at step = warmup
    assert abs(orc.inverse_sqrt_lr(4000, 1024) - 1024 ** -0.5 * 4000 ** -0.5) < 1e-18
    assert abs(orc.inverse_sqrt_lr(1, 1024) - 1024 ** -0.5 * 4000 ** -1.5) < 1e-18
    assert orc.inverse_sqrt_lr(3999, 1024) < orc.inverse_sqrt_lr(4000, 1024) > orc.inverse_sqrt_lr(4001, 1024)


# ------------------------------------------------------------------ workload generators

def test_generators_are_seeded_and_shaped():
    w = wl.CONFIGS["cfg1"]
    a = wl.draw_params(w)
    b = wl.draw_params(w)
    assert all(np.array_equal(a[k], b[k]) for k in a)
    assert abs(float(a["c0.l0.mlp.w1"].std()) - 0.02) < 2e-3
    assert abs(float(a["c0.l0.ln1.g"].mean()) - 1.0) < 1e-2
    tok, tgt = wl.draw_tokens(w)
    assert tok.shape == (w.B, w.T) and tgt.shape == (w.B, w.T)
    assert np.array_equal(tok[:, 1:], tgt[:, :-1])          # next-token targets
    assert tok.min() >= 0 and tok.max() < w.V
    z = wl.CONFIGS["cfg2"].with_(B=64, T=256)
    tz, _ = wl.draw_tokens(z)
    # Zipf(1.1): rank-1 token has probability 1/sum r^-1.1 ~= 0.1 over 50257 ranks
    p1 = 1.0 / np.sum(np.arange(1, z.V + 1, dtype=np.float64) ** -1.1)
    assert abs((tz == 0).mean() - p1) < 0.01
    # per block 12 d^2 matrix weights (4d^2 attention + 8d^2 MLP at F = 4d) + 13 d vector entries
    w4 = wl.CONFIGS["cfg4"]
    per_block = sum(int(np.prod(s)) for nme, _, _, s in wl.tensor_specs(w4) if nme.startswith("c0.l0."))
    assert per_block == 12 * w4.d ** 2 + 13 * w4.d


# ------------------------------------------------------------------ the paper's own head weightings

def _rule_window_loss(P, tok, tgt, w, k, n, rule):
    """Independent formula: the scalar whose plain derivative w.r.t. component k's parameters the rule asks for."""
    L = orc.head_losses(P, tok, tgt, w.K, w.Lc, w.H)
    far = min(k + n - 1, w.K - 1)
    if rule == "far":
        return L[far]
    return 0.5 * L[k] + 0.5 * L[far]


@pytest.mark.parametrize("rule", ["far", "mean"])
@pytest.mark.parametrize("n", [2, 3])
def test_paper_rules_finite_differences(rule, n):
    """Sec. 3: module k updated from L_{k+N-1} ("far"), or from the mean of L_k and L_{k+N-1} ("mean")."""
    w = TINY
    P, tok, tgt = _setup(w)
    _, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n, rule=rule)
    rng = np.random.default_rng(100 + n)
    for name, comp, is_head, shape in wl.tensor_specs(w):
        size = int(np.prod(shape))
        for _ in range(2):
            flat = int(rng.integers(0, size))
            idx = np.unravel_index(flat, shape)
            if name == "wte":
                idx = (int(tok.reshape(-1)[flat % tok.size]), idx[1])
            if is_head:
                fn = lambda: orc.head_losses(P, tok, tgt, w.K, w.Lc, w.H)[comp]
            else:
                fn = lambda: _rule_window_loss(P, tok, tgt, w, comp, n, rule)
            fd = _fd(P, name, idx, fn)
            g = G[name][idx]
            assert abs(fd - g) / max(abs(fd), abs(g), 1e-7) < 1e-6, (name, idx, fd, g)


def test_paper_rules_relations():
    w = TINY2
    P, tok, tgt = _setup(w)
    specs = wl.tensor_specs(w)
    G = {(r, n): orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n, rule=r)[1]
         for r in ("sum", "far", "mean") for n in (1, 2, w.K)}
    for name, comp, is_head, _ in specs:
        # n = 1: the three rules coincide (local learning)
        assert np.array_equal(G[("far", 1)][name], G[("sum", 1)][name])
        assert np.array_equal(G[("mean", 1)][name], G[("sum", 1)][name])
        # head parameters never depend on the rule
        if is_head:
            assert np.array_equal(G[("far", 2)][name], G[("sum", 2)][name])
            continue
        # n = 2: the mean of the two heads is half their sum, except in the top component (one head only)
        if comp < w.K - 1:
            assert np.allclose(G[("mean", 2)][name], 0.5 * G[("sum", 2)][name], rtol=1e-12, atol=1e-15), name
        else:
            assert np.allclose(G[("mean", 2)][name], G[("sum", 2)][name], rtol=1e-12, atol=1e-15), name
    # "far" with n = K is end-to-end training of the final loss alone (Sec. 3: N = number of modules)
    Pt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in P.items()}
    tt = torch.tensor(tok.reshape(-1), dtype=torch.long)
    yy = torch.tensor(tgt.reshape(-1), dtype=torch.long)
    x = Pt["wte"][tt] + Pt["wpe"][torch.arange(w.T).repeat(w.B)]
    x = _torch_forward_from(Pt, x, 0, w.K, w)
    u = Fnn.layer_norm(x, (w.d,), Pt[f"head{w.K - 1}.ln.g"], Pt[f"head{w.K - 1}.ln.b"], eps=1e-5)
    Fnn.cross_entropy(Fnn.linear(u, Pt[f"head{w.K - 1}.w"]), yy).backward()
    for name, comp, is_head, _ in specs:
        if not is_head:
            assert np.allclose(G[("far", w.K)][name], Pt[name].grad.numpy(), rtol=1e-9, atol=1e-13), name


@pytest.mark.parametrize("rule", ["sum", "far", "mean"])
@pytest.mark.parametrize("head_layers", [0, 1])
def test_bounded_memory_step_equals_the_plain_one(rule, head_layers):
    """nwise_gradients_bounded (boundaries kept, blocks recomputed, gradients emitted when final, heads from the
    top down) gives the losses and gradients of nwise_gradients for every n: same passes, other bookkeeping."""
    import workloads as wl
    w = wl.Workload("bnd", K=3, Lc=2, d=8, H=2, F=16, V=11, T=5, B=2, n=1, zipf=False, Lh=head_layers)
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    for n in (1, 2, 3):
        l0, G0 = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n, rule=rule, head_layers=head_layers)
        got = {}
        order = []

        def emit(name, g):
            assert name not in got
            got[name] = np.array(g, dtype=np.float64, copy=True)
            order.append(name)

        l1 = orc.nwise_gradients_bounded(P, tok, tgt, w.K, w.Lc, w.H, n, emit, rule=rule, head_layers=head_layers)
        assert np.allclose(l0, l1, rtol=1e-13, atol=0)
        assert set(got) == set(G0)
        for name in G0:
            assert np.allclose(got[name], G0[name], rtol=1e-10, atol=1e-15), (n, name)
        # a component's tensors are emitted only after its own head has been processed, i.e. after every head above
        assert order.index("head2.w") < order.index("c2.l0.mlp.w1") < order.index("head1.w") < order.index("c1.l0.mlp.w1")
