"""fp64 CPU oracle for one n-wise interlocking-backpropagation training step.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
training step computes; it exists to check the CUDA library and is never on the
product path.  It shares no code with the CUDA sources and imports nothing from
the package.  Everything is numpy in float64; `@` (matmul) is used as a library
step, nothing is fused, tiled or reordered beyond processing independent token
rows of a head in blocks to bound host memory.

What it follows
---------------
* Network = composition of K contiguous groups of layers ("modules", here
  components), Sec. 3: f = f_cK o ... o f_c1.  Each component is Lc pre-LN
  GPT-2-style Transformer blocks (Sec. 4.3 says the model largely follows GPT-2).
* Auxiliary network h_ck after every component and the local loss
  L_ck(x, y) = L(h_ck(f_ck o ... o f_c1 (x)), y), Sec. 3 (unnumbered equations);
  L is the mean next-token cross-entropy.  The auxiliary network here is
  LayerNorm followed by an untied linear map to the vocabulary; with
  head_layers > 0 that many Transformer blocks come first, which is the
  auxiliary network of the paper's Transformer runs (App. B.3).
* Micro-batching (Sec. 3.1): nwise_gradients_microbatched averages the
  gradients of equal groups of sequences before the single update.
* n-wise rule, Sec. 3 and Fig. 2: the gradient of head h flows through its own
  component and across n-1 component boundaries, then stops.  Reading used here:
  the gradients of all heads whose window covers a component are summed with
  weight one, so for parameters of component k (1-based)
      G(theta_ck) = d/d theta_ck  sum_{h=k}^{min(k+n-1, K)} L_h ,
  head parameters receive only their own loss's gradient, and the embeddings
  belong to component 1.  n = 1 is local learning; n = K is ordinary
  backpropagation of sum_k L_k.
* Optimiser: Adam with the hyper-parameters of App. B.3, written as AdamW
  (decoupled weight decay; weight decay 0 gives the paper's Adam).

Pins (tests/test_oracle_pins.py, tests/test_oracle_aux_blocks.py): central finite differences of the windowed loss
sums on tiny nets, brute-force softmax/attention/cross-entropy on tiny inputs,
the locality / nesting / n=K invariants of the rule, ln(V) for a zero-weight
head, causal-mask independence, closed-form first AdamW step.  No numeric
value printed in the paper exists for this path (its Transformer results are
only in figures), so parity with the paper's own runs is unpinned; parity with
the rule as stated above is pinned by the tests listed.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64
LN_EPS = 1e-5


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=F64)


# ----------------------------------------------------------------------------
# Elementary pieces (textbook definitions)
# ----------------------------------------------------------------------------

def layernorm_fwd(x: np.ndarray, g: np.ndarray, b: np.ndarray, eps: float = LN_EPS):
    """y = g * (x - mean) / sqrt(var + eps) + b, biased variance over the last axis."""
    mu = x.mean(axis=-1, keepdims=True)
    xc = x - mu
    var = (xc * xc).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = xc * rstd
    return xhat * g + b, (xhat, rstd)


def layernorm_bwd(dy: np.ndarray, cache, g: np.ndarray):
    """Derivative of layernorm_fwd: returns (dx, dg, db)."""
    xhat, rstd = cache
    dg = (dy * xhat).sum(axis=0)
    db = dy.sum(axis=0)
    dxhat = dy * g
    m1 = dxhat.mean(axis=-1, keepdims=True)
    m2 = (dxhat * xhat).mean(axis=-1, keepdims=True)
    dx = (dxhat - m1 - xhat * m2) * rstd
    return dx, dg, db


_GELU_C = math.sqrt(2.0 / math.pi)


def gelu(x: np.ndarray) -> np.ndarray:
    """tanh form of GELU (GPT-2): 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))."""
    return 0.5 * x * (1.0 + np.tanh(_GELU_C * (x + 0.044715 * x ** 3)))


def gelu_grad(x: np.ndarray) -> np.ndarray:
    u = _GELU_C * (x + 0.044715 * x ** 3)
    t = np.tanh(u)
    du = _GELU_C * (1.0 + 3.0 * 0.044715 * x * x)
    return 0.5 * (1.0 + t) + 0.5 * x * (1.0 - t * t) * du


def _split_heads(a: np.ndarray, B: int, T: int, H: int) -> np.ndarray:
    """[B*T, H*dh] -> [B, H, T, dh]"""
    dh = a.shape[1] // H
    return a.reshape(B, T, H, dh).transpose(0, 2, 1, 3)


def _merge_heads(a: np.ndarray) -> np.ndarray:
    """[B, H, T, dh] -> [B*T, H*dh]"""
    B, H, T, dh = a.shape
    return a.transpose(0, 2, 1, 3).reshape(B * T, H * dh)


def _causal_probs(q: np.ndarray, k: np.ndarray) -> np.ndarray:
    """softmax over keys j <= i of q_i . k_j / sqrt(dh);  [B,H,T,T]."""
    dh = q.shape[-1]
    T = q.shape[-2]
    s = (q @ k.transpose(0, 1, 3, 2)) / math.sqrt(dh)
    mask = np.triu(np.ones((T, T), dtype=bool), k=1)
    s = np.where(mask, -np.inf, s)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    return p / p.sum(axis=-1, keepdims=True)


def attention_fwd(qkv: np.ndarray, B: int, T: int, H: int) -> np.ndarray:
    """Causal multi-head self-attention on packed [Ntok, 3d] = [Q | K | V]."""
    d = qkv.shape[1] // 3
    q = _split_heads(qkv[:, :d], B, T, H)
    k = _split_heads(qkv[:, d:2 * d], B, T, H)
    v = _split_heads(qkv[:, 2 * d:], B, T, H)
    p = _causal_probs(q, k)
    return _merge_heads(p @ v)


def attention_bwd(do: np.ndarray, qkv: np.ndarray, B: int, T: int, H: int) -> np.ndarray:
    """Gradient of attention_fwd w.r.t. the packed qkv (probabilities recomputed)."""
    d = qkv.shape[1] // 3
    dh = d // H
    q = _split_heads(qkv[:, :d], B, T, H)
    k = _split_heads(qkv[:, d:2 * d], B, T, H)
    v = _split_heads(qkv[:, 2 * d:], B, T, H)
    p = _causal_probs(q, k)
    dO = _split_heads(do, B, T, H)
    dv = p.transpose(0, 1, 3, 2) @ dO
    dp = dO @ v.transpose(0, 1, 3, 2)
    ds = p * (dp - (dp * p).sum(axis=-1, keepdims=True))
    ds = ds / math.sqrt(dh)
    dq = ds @ k
    dk = ds.transpose(0, 1, 3, 2) @ q
    return np.concatenate([_merge_heads(dq), _merge_heads(dk), _merge_heads(dv)], axis=1)


# ----------------------------------------------------------------------------
# Transformer block, component, embedding, head
# ----------------------------------------------------------------------------

def block_fwd(x: np.ndarray, P: Dict[str, np.ndarray], pre: str, B: int, T: int, H: int):
    """Pre-LN block: x += Wo Attn(Wqkv LN1 x);  x += W2 GELU(W1 LN2 x)."""
    c = {"x0": x}
    y1, c["ln1"] = layernorm_fwd(x, _f64(P[pre + "ln1.g"]), _f64(P[pre + "ln1.b"]))
    c["y1"] = y1
    qkv = y1 @ _f64(P[pre + "attn.wqkv"]).T + _f64(P[pre + "attn.bqkv"])
    c["qkv"] = qkv
    o = attention_fwd(qkv, B, T, H)
    c["o"] = o
    x1 = x + o @ _f64(P[pre + "attn.wo"]).T + _f64(P[pre + "attn.bo"])
    y2, c["ln2"] = layernorm_fwd(x1, _f64(P[pre + "ln2.g"]), _f64(P[pre + "ln2.b"]))
    c["y2"] = y2
    hpre = y2 @ _f64(P[pre + "mlp.w1"]).T + _f64(P[pre + "mlp.b1"])
    c["hpre"] = hpre
    hact = gelu(hpre)
    c["hact"] = hact
    x2 = x1 + hact @ _f64(P[pre + "mlp.w2"]).T + _f64(P[pre + "mlp.b2"])
    return x2, c


def block_bwd(dx2: np.ndarray, c, P, pre: str, B: int, T: int, H: int, G: Dict[str, np.ndarray]):
    """Back-propagate dx2 through one block; parameter gradients are ADDED into G."""
    def acc(name, val):
        G[name] = G[name] + val if name in G else val

    # MLP branch
    acc(pre + "mlp.b2", dx2.sum(axis=0))
    acc(pre + "mlp.w2", dx2.T @ c["hact"])
    dhact = dx2 @ _f64(P[pre + "mlp.w2"])
    dhpre = dhact * gelu_grad(c["hpre"])
    acc(pre + "mlp.b1", dhpre.sum(axis=0))
    acc(pre + "mlp.w1", dhpre.T @ c["y2"])
    dy2 = dhpre @ _f64(P[pre + "mlp.w1"])
    dx1_ln, dg, db = layernorm_bwd(dy2, c["ln2"], _f64(P[pre + "ln2.g"]))
    acc(pre + "ln2.g", dg)
    acc(pre + "ln2.b", db)
    dx1 = dx2 + dx1_ln
    # attention branch
    acc(pre + "attn.bo", dx1.sum(axis=0))
    acc(pre + "attn.wo", dx1.T @ c["o"])
    do = dx1 @ _f64(P[pre + "attn.wo"])
    dqkv = attention_bwd(do, c["qkv"], B, T, H)
    acc(pre + "attn.bqkv", dqkv.sum(axis=0))
    acc(pre + "attn.wqkv", dqkv.T @ c["y1"])
    dy1 = dqkv @ _f64(P[pre + "attn.wqkv"])
    dx0_ln, dg, db = layernorm_bwd(dy1, c["ln1"], _f64(P[pre + "ln1.g"]))
    acc(pre + "ln1.g", dg)
    acc(pre + "ln1.b", db)
    return dx1 + dx0_ln


def embed_fwd(tokens: np.ndarray, P) -> np.ndarray:
    """a_0[i] = wte[token_i] + wpe[position_i];  tokens [B,T] -> [B*T, d]."""
    B, T = tokens.shape
    wte = _f64(P["wte"])
    wpe = _f64(P["wpe"])
    x = wte[tokens.reshape(-1)] + np.tile(wpe[:T], (B, 1))
    return x


def embed_bwd(dx: np.ndarray, tokens: np.ndarray, P, G):
    B, T = tokens.shape
    dwte = np.zeros(P["wte"].shape, dtype=F64)
    np.add.at(dwte, tokens.reshape(-1), dx)
    dwpe = np.zeros(P["wpe"].shape, dtype=F64)
    dwpe[:T] = dx.reshape(B, T, -1).sum(axis=0)
    G["wte"] = G["wte"] + dwte if "wte" in G else dwte
    G["wpe"] = G["wpe"] + dwpe if "wpe" in G else dwpe


def component_fwd(x: np.ndarray, P, k: int, Lc: int, B: int, T: int, H: int):
    caches = []
    for l in range(Lc):
        x, c = block_fwd(x, P, f"c{k}.l{l}.", B, T, H)
        caches.append(c)
    return x, caches


def component_bwd(dx: np.ndarray, caches, P, k: int, B: int, T: int, H: int, G):
    for l in reversed(range(len(caches))):
        dx = block_bwd(dx, caches[l], P, f"c{k}.l{l}.", B, T, H, G)
    return dx


def head_loss(a: np.ndarray, targets: np.ndarray, P, k: int, want_grad: bool, row_block: int = 1024,
              head_layers: int = 0, B: int = 0, T: int = 0, H: int = 0):
    """Auxiliary head k: z = LN(t(a)) W^T, L = mean_i (logsumexp_v z_iv - z_i,y_i).

    t is the identity for head_layers = 0 (LayerNorm + linear head).  For head_layers > 0 it is that many
    pre-LN Transformer blocks of the main network's shape with parameters head{k}.l{j}.* — the auxiliary
    network of the paper's Transformer runs (App. B.3: main network output -> 2 Transformer blocks ->
    embedding matrix -> logits; the LayerNorm before the matrix is this build's, as pre-LN blocks need one).
    B, T, H are needed by the blocks' attention only.

    Returns (loss, da, grads dict) — the last two None unless want_grad.
    Rows are independent, so they are processed in blocks to bound memory.
    """
    g = _f64(P[f"head{k}.ln.g"])
    b = _f64(P[f"head{k}.ln.b"])
    W = _f64(P[f"head{k}.w"])
    y = targets.reshape(-1)
    N = a.shape[0]
    hcaches = []
    for j in range(head_layers):
        a, c = block_fwd(a, P, f"head{k}.l{j}.", B, T, H)
        hcaches.append(c)
    u, cache = layernorm_fwd(a, g, b)
    loss = 0.0
    du = np.zeros_like(u) if want_grad else None
    dW = np.zeros_like(W) if want_grad else None
    for r0 in range(0, N, row_block):
        r1 = min(N, r0 + row_block)
        z = u[r0:r1] @ W.T
        zmax = z.max(axis=1, keepdims=True)
        ez = np.exp(z - zmax)
        se = ez.sum(axis=1, keepdims=True)
        lse = (zmax + np.log(se))[:, 0]
        rows = np.arange(r1 - r0)
        loss += float((lse - z[rows, y[r0:r1]]).sum())
        if want_grad:
            dz = ez / se
            dz[rows, y[r0:r1]] -= 1.0
            dz /= N
            dW += dz.T @ u[r0:r1]
            du[r0:r1] = dz @ W
    loss /= N
    if not want_grad:
        return loss, None, None
    da, dg, db = layernorm_bwd(du, cache, g)
    hg = {f"head{k}.ln.g": dg, f"head{k}.ln.b": db, f"head{k}.w": dW}
    for j in reversed(range(head_layers)):
        da = block_bwd(da, hcaches[j], P, f"head{k}.l{j}.", B, T, H, hg)
    return loss, da, hg


# ----------------------------------------------------------------------------
# The training step
# ----------------------------------------------------------------------------

def forward_all(P, tokens: np.ndarray, K: int, Lc: int, H: int):
    """a_0 .. a_K and the per-component caches."""
    B, T = tokens.shape
    a = [embed_fwd(tokens, P)]
    caches = []
    for k in range(K):
        x, c = component_fwd(a[-1], P, k, Lc, B, T, H)
        a.append(x)
        caches.append(c)
    return a, caches


def head_losses(P, tokens, targets, K: int, Lc: int, H: int, head_layers: int = 0) -> List[float]:
    B, T = tokens.shape
    a, _ = forward_all(P, tokens, K, Lc, H)
    return [head_loss(a[k + 1], targets, P, k, False, head_layers=head_layers, B=B, T=T, H=H)[0] for k in range(K)]


def head_weight(k: int, h: int, n: int, K: int, rule: str) -> float:
    """Weight of head h's gradient in the update of component k's parameters (0-based, k <= h <= k+n-1).

    "sum"  : every head whose window covers the component counts once (the reading this build targets).
    "far"  : the paper's main-text rule (Sec. 3): module k is updated from L_{c_{k+N-1}} alone; the window is
             clamped at the last head, which makes N = number of modules end-to-end training of the final loss.
    "mean" : the variant of the paper's Transformer experiments (Sec. 3, App. B.3): the mean of the
             gradients from the module's own head and from head k+N-1.
    """
    far = min(k + n - 1, K - 1)
    if rule == "sum":
        return 1.0
    if rule == "far":
        return 1.0 if h == far else 0.0
    if rule == "mean":
        return 0.5 * (h == k) + 0.5 * (h == far)
    raise ValueError("rule must be 'sum', 'far' or 'mean'")


def nwise_gradients(P, tokens: np.ndarray, targets: np.ndarray, K: int, Lc: int, H: int, n: int,
                    head_weights: Optional[Sequence[float]] = None, rule: str = "sum", head_layers: int = 0):
    """One n-wise step's losses and parameter "gradients" (Sec. 3, Fig. 2).

    For every head h (0-based here) its loss is back-propagated through the head
    and then through components h, h-1, ..., max(h-n+1, 0); the gradient is dropped
    at the input of the last of these (the stop at the component boundary).  Each
    head is a separate backward pass; the parameter gradients it leaves in component k
    enter the result with weight head_weight(k, h, n, K, rule) (all 1 for rule "sum").
    Head parameters always receive their own loss's gradient with weight 1; the
    embeddings belong to component 0.
    head_weights (default all 1) scales each head's loss before back-propagation.
    head_layers > 0 puts that many Transformer blocks inside every auxiliary head (see head_loss); they are
    head parameters and so receive only their own loss's gradient.
    """
    if not (1 <= n <= K):
        raise ValueError("n must be in [1, K]")
    B, T = tokens.shape
    a, caches = forward_all(P, tokens, K, Lc, H)
    losses: List[float] = []
    G: Dict[str, np.ndarray] = {}
    for h in range(K):
        loss, da, hg = head_loss(a[h + 1], targets, P, h, True, head_layers=head_layers, B=B, T=T, H=H)
        losses.append(loss)
        wgt = 1.0 if head_weights is None else float(head_weights[h])
        for name, val in hg.items():
            G[name] = val * wgt
        dx = da * wgt
        lowest = max(h - n + 1, 0)
        for k in range(h, lowest - 1, -1):
            wk = head_weight(k, h, n, K, rule)
            if wk == 1.0:
                dx = component_bwd(dx, caches[k], P, k, B, T, H, G)
            else:
                Gk: Dict[str, np.ndarray] = {}
                dx_in = component_bwd(dx, caches[k], P, k, B, T, H, Gk)
                if k == 0:
                    embed_bwd(dx_in, tokens, P, Gk)
                if wk != 0.0:
                    for name, val in Gk.items():
                        G[name] = G[name] + wk * val if name in G else wk * val
                dx = dx_in
                continue
            if k == 0:
                embed_bwd(dx, tokens, P, G)
        # below `lowest` dx is the gradient at a stopped boundary and is discarded.
    for name in P:
        if name not in G:
            G[name] = np.zeros(P[name].shape, dtype=F64)
    return losses, G


def nwise_gradients_bounded(P, tokens: np.ndarray, targets: np.ndarray, K: int, Lc: int, H: int, n: int, emit,
                            rule: str = "sum", head_layers: int = 0) -> List[float]:
    """The step of nwise_gradients with bounded memory, for configurations whose intermediate values do not fit
    the host (the arithmetic of every pass is the same; only what is kept, and for how long, differs).

    * The forward pass keeps the K+1 boundary activations only; the blocks' intermediate values of a component are
      recomputed (component_fwd from its stored input) each time a head's backward pass reaches it.
    * Heads are taken from the top down.  Component k receives gradient from heads k .. k+n-1 (Sec. 3), so once head k
      has been processed its parameter gradients are final: they are handed to emit(name, gradient) and dropped.
      Head parameters are final right after their own pass.  Tensors that never received a gradient are emitted
      as zeros.
    Returns the K head losses.  A test pins it to nwise_gradients on small nets for every n and rule.
    """
    if not (1 <= n <= K):
        raise ValueError("n must be in [1, K]")
    B, T = tokens.shape
    a = [embed_fwd(tokens, P)]
    for k in range(K):
        x, _ = component_fwd(a[-1], P, k, Lc, B, T, H)
        a.append(x)
    losses: List[float] = [0.0] * K
    G: Dict[str, np.ndarray] = {}
    emitted = set()

    def flush(prefixes):
        for name in list(G.keys()):
            if any(name == p or name.startswith(p) for p in prefixes):
                emit(name, G.pop(name))
                emitted.add(name)

    for h in reversed(range(K)):
        loss, da, hg = head_loss(a[h + 1], targets, P, h, True, head_layers=head_layers, B=B, T=T, H=H)
        losses[h] = loss
        for name, val in hg.items():
            emit(name, val)
            emitted.add(name)
        del hg
        dx = da
        lowest = max(h - n + 1, 0)
        for k in range(h, lowest - 1, -1):
            _, caches_k = component_fwd(a[k], P, k, Lc, B, T, H)
            wk = head_weight(k, h, n, K, rule)
            if wk == 1.0:
                dx = component_bwd(dx, caches_k, P, k, B, T, H, G)
                if k == 0:
                    embed_bwd(dx, tokens, P, G)
            else:
                Gk: Dict[str, np.ndarray] = {}
                dx = component_bwd(dx, caches_k, P, k, B, T, H, Gk)
                if k == 0:
                    embed_bwd(dx, tokens, P, Gk)
                if wk != 0.0:
                    for name, val in Gk.items():
                        G[name] = G[name] + wk * val if name in G else wk * val
                del Gk
            del caches_k
        # every head whose window covers component h has now been processed
        flush([f"c{h}."] + (["wte", "wpe"] if h == 0 else []))
    for name in P:
        if name not in emitted:
            emit(name, np.zeros(P[name].shape, dtype=F64))
    return [float(x) for x in losses]


def nwise_gradients_microbatched(P, tokens: np.ndarray, targets: np.ndarray, K: int, Lc: int, H: int, n: int,
                                 micro_batches: int, rule: str = "sum", head_layers: int = 0):
    """The same step with the mini-batch split into `micro_batches` equal groups of sequences (Sec. 3.1:
    micro-batching as in pipeline parallelism): every group is a separate forward/backward, the parameter
    gradients of the groups are averaged and one update follows.  Returns (mean losses, gradients).
    With equal group sizes this is the gradient of the whole mini-batch; a test pins that identity."""
    Bfull = tokens.shape[0]
    if micro_batches < 1 or Bfull % micro_batches:
        raise ValueError("the batch must split into equal micro-batches")
    per = Bfull // micro_batches
    losses = np.zeros(K, dtype=F64)
    G: Dict[str, np.ndarray] = {}
    for mb in range(micro_batches):
        sl = slice(mb * per, (mb + 1) * per)
        l, g = nwise_gradients(P, tokens[sl], targets[sl], K, Lc, H, n, rule=rule, head_layers=head_layers)
        losses += np.asarray(l, dtype=F64) / micro_batches
        for name, val in g.items():
            G[name] = G[name] + val / micro_batches if name in G else val / micro_batches
    return [float(x) for x in losses], G


def adamw_step(P: Dict[str, np.ndarray], G: Dict[str, np.ndarray], state: Dict[str, Tuple[np.ndarray, np.ndarray]],
               step: int, lr: float, beta1: float = 0.9, beta2: float = 0.98, eps: float = 1e-9,
               weight_decay: float = 0.0) -> Dict[str, np.ndarray]:
    """AdamW update number `step` (1-based).  Returns new fp64 parameters; updates state in place.

    m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;  mhat = m/(1-b1^t);  vhat = v/(1-b2^t);
    p <- p - lr (mhat / (sqrt(vhat) + eps) + wd p), the decay applied to tensors of rank 2 only.
    Defaults are the paper's Adam settings (App. B.3).
    """
    out = {}
    for name, p in P.items():
        p = _f64(p)
        g = _f64(G[name])
        m, v = state.get(name, (np.zeros_like(p), np.zeros_like(p)))
        m = beta1 * m + (1.0 - beta1) * g
        v = beta2 * v + (1.0 - beta2) * g * g
        state[name] = (m, v)
        mhat = m / (1.0 - beta1 ** step)
        vhat = v / (1.0 - beta2 ** step)
        wd = weight_decay if p.ndim == 2 else 0.0
        out[name] = p - lr * (mhat / (np.sqrt(vhat) + eps) + wd * p)
    return out


def inverse_sqrt_lr(step: int, d_model: int, warmup: int = 4000) -> float:
    """Learning-rate schedule of App. B.3: d^-0.5 min(step^-0.5, step warmup^-1.5)."""
    return d_model ** -0.5 * min(step ** -0.5, step * warmup ** -1.5)
