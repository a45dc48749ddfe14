"""Error paths, determinism and the pipeline placement of the CUDA library (GPU).  Nothing here faults, traps or
hangs the device: the expired wait is a kernel that gives up after a millisecond and returns, the failing
allocation is the caller's own allocator hook returning NULL, and the out-of-range head is ordinary arithmetic."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import workloads as wl
from oracle import il_oracle as orc
from paper_2010_04116_b200 import ILError, Model
from paper_2010_04116_b200 import binding as il

pytestmark = pytest.mark.gpu
HP = dict(lr=1e-3, beta1=0.9, beta2=0.98, eps=1e-9, weight_decay=0.01)


def _small(n=2, **kw):
    w = wl.CONFIGS["cfg1"]
    m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, n, w.B, w.T, **kw)
    P = wl.draw_params(w)
    m.set_params(P)
    tok, tgt = wl.draw_tokens(w)
    return w, m, P, tok, tgt


def test_expired_device_wait_is_reported_and_the_next_step_is_clean():
    """A bounded wait that runs out (1 ms, on a barrier nobody arrives at) sets the model's error word; il_sync
    returns IL_ERR_TIMEOUT and clears it; the step after that matches the oracle."""
    w, m, P, tok, tgt = _small()
    try:
        m.train_step(tok, tgt)
        m.sync()
        il.op_wait_probe(m.error_word(0), 1000, m.streams[0].cuda_stream)
        with pytest.raises(ILError) as e:
            m.sync()
        assert e.value.status == 5 and "IL_ERR_TIMEOUT" in str(e.value)
        word = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        il.op_wait_probe(word.data_ptr(), 500)
        torch.cuda.synchronize()
        assert int(word.item()) in (1, 2, 3)          # a DEV_TIMEOUT_* code
        m.sync()                                       # cleared by the report: no error now
        m.train_step(tok, tgt)
        losses = m.get_losses()
        m.sync()
        ol, OG = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, 2)
        assert np.all(np.abs(losses - np.array(ol)) <= 1e-3 * np.abs(np.array(ol)))
        g = m.get_grad("c0.l0.mlp.w1").astype(np.float64)
        assert np.linalg.norm(g - OG["c0.l0.mlp.w1"]) / np.linalg.norm(OG["c0.l0.mlp.w1"]) < 2e-2
    finally:
        m.close()


def test_update_is_skipped_while_the_error_word_is_set():
    """A step whose head left the exp(logit) range must not reach the parameters: AdamW leaves weights, moments and
    the step counter as they were, il_sync says IL_ERR_NONFINITE, and training continues after the cause is gone."""
    w, m, P, tok, tgt = _small(n=1)
    try:
        m.train_step(tok, tgt, adamw=HP)
        m.sync()
        names = ["c0.l0.mlp.w1", "c1.l1.attn.wqkv", "head0.w", "head1.ln.g", "wte"]
        before = {nm: (m.get_param(nm), *m.get_opt_state(nm)) for nm in names}
        assert before[names[0]][3] == 1
        good = {nm: m.get_param(nm) for nm in ("head0.w", "head1.w")}
        for nm in good:                                  # both heads out of range: every component skips
            m.set_param(nm, (good[nm] * 4000.0).astype(np.float32))
        before["head0.w"] = (m.get_param("head0.w"), *m.get_opt_state("head0.w"))
        with pytest.raises(ILError) as e:
            m.train_step(tok, tgt, adamw=HP)
            m.sync()
        assert e.value.status == 6
        assert "0 of 1 optimiser updates" in str(e.value)
        for nm in names:
            p, mm, vv, step = before[nm]
            assert np.array_equal(m.get_param(nm), p), nm
            m2, v2, s2 = m.get_opt_state(nm)
            assert np.array_equal(m2, mm) and np.array_equal(v2, vv) and s2 == 1, nm
        for nm in good:
            m.set_param(nm, good[nm])
        m.train_step(tok, tgt, adamw=HP)
        m.sync()
        assert m.get_opt_state("c0.l0.mlp.w1")[2] == 2
        assert not np.array_equal(m.get_param("c0.l0.mlp.w1"), before["c0.l0.mlp.w1"][0])
    finally:
        m.close()


def test_recompute_head_has_no_logit_range_limit():
    w, m, P, tok, tgt = _small(n=1, head_mode="recompute")
    try:
        m.set_param("head0.w", (P["head0.w"] * 4000.0).astype(np.float32))
        m.train_step(tok, tgt)
        m.sync()
        assert np.all(np.isfinite(m.get_grad("head0.w")))
        P2 = dict(P)
        P2["head0.w"] = (P["head0.w"] * 4000.0).astype(np.float32)
        ol, OG = orc.nwise_gradients(P2, tok, tgt, w.K, w.Lc, w.H, 1)
        assert np.all(np.abs(m.get_losses() - np.array(ol)) <= 1e-3 * np.abs(np.array(ol)))
    finally:
        m.close()


def test_stored_head_falls_back_to_recomputation_when_a_row_leaves_its_range():
    """The stored-exp(logit) head reports a row outside [-80, 80] and the model switches to the recomputing head
    (which has no such limit) for all later steps: the repeated step succeeds, and gives bit for bit what a model
    created in recompute mode gives (same chunking, same kernels)."""
    w, m, P, tok, tgt = _small(n=2, attn_bwd="two_kernels")           # every sum of these sizes in a fixed order
    _, m2, _, _, _ = _small(n=2, head_mode="recompute", attn_bwd="two_kernels")
    try:
        bad = (P["head0.w"] * 4000.0).astype(np.float32)
        assert m.head_mode == "stored" and m2.head_mode == "recompute"
        m.set_param("head0.w", bad)
        m2.set_param("head0.w", bad)
        with pytest.raises(ILError) as e:
            m.train_step(tok, tgt, adamw=HP)
            m.sync()
        assert e.value.status == 6 and "IL_HEAD_RECOMPUTE" in str(e.value)
        assert m.head_mode == "recompute"
        assert m.get_opt_state("head1.w")[2] == 0            # nothing was applied
        m.train_step(tok, tgt)                                # the same step again, same parameters
        losses = m.get_losses()
        m.sync()
        m2.train_step(tok, tgt)
        losses2 = m2.get_losses()
        m2.sync()
        assert np.array_equal(losses, losses2)
        for nm in ("head0.w", "head1.w", "c0.l0.mlp.w1", "c1.l1.attn.wqkv"):
            g = m.get_grad(nm)
            assert np.all(np.isfinite(g)) and np.array_equal(g, m2.get_grad(nm)), nm
    finally:
        m.close()
        m2.close()


def test_allocator_returning_null_gives_oom_and_everything_is_handed_back():
    w = wl.CONFIGS["cfg1"]
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    base = torch.cuda.memory_allocated()
    probe = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, w.B, w.T)
    total_calls = probe._alloc_calls
    probe.close()
    assert total_calls > 20
    for fail_at in (0, 3, total_calls // 2, total_calls - 1):
        with pytest.raises(ILError) as e:
            Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, w.B, w.T, alloc_fail_at=fail_at)
        assert e.value.status == 3, fail_at
        assert torch.cuda.memory_allocated() <= base, fail_at
    m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, w.B, w.T)       # and the next creation succeeds
    m.close()
    assert torch.cuda.memory_allocated() <= base


def test_growing_n_hands_back_the_superseded_scratch():
    w = wl.Workload("k4s", K=4, Lc=1, d=128, H=2, F=256, V=300, T=64, B=2, n=1, zipf=True)
    a = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 1, w.B, w.T)
    b = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, w.B, w.T)
    try:
        small, big = a.stats()[0], b.stats()[0]
        assert big > small
        a.set_n(2)
        assert a.stats()[0] == big
        a.set_n(1)
        a.set_n(3)
        assert a.stats()[0] == big                      # n = 3 needs the same two stacked streams at K = 4
    finally:
        a.close()
        b.close()


def test_checkpoint_resume_gives_the_identical_next_update():
    """Parameters, Adam moments and the step counter moved to a fresh model give the same second update
    (compared on tensors whose gradients are summed in a fixed order; the others within 1e-6)."""
    w, m, P, tok, tgt = _small(attn_bwd="two_kernels")
    tok2, tgt2 = wl.draw_tokens(w, step=1)
    m2 = None
    try:
        m.train_step(tok, tgt, adamw=HP)
        m.sync()
        m2 = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, w.B, w.T, attn_bwd="two_kernels")
        for nm in m.names:
            m2.set_param(nm, m.get_param(nm))
            mm, vv, step = m.get_opt_state(nm)
            m2.set_opt_state(nm, mm, vv, step)
        for mdl in (m, m2):
            mdl.train_step(tok2, tgt2, adamw=HP)
            mdl.sync()
        for nm in m.names:
            a, b = m.get_param(nm), m2.get_param(nm)
            assert m2.get_opt_state(nm)[2] == 2
            if nm.endswith(".w") or nm in ("wte", "wpe") or nm.endswith("wqkv") or nm.endswith("wo") \
                    or nm.endswith("w1") or nm.endswith("w2"):
                assert np.array_equal(a, b), nm
            else:
                assert np.max(np.abs(a - b)) < 1e-6, nm
    finally:
        m.close()
        if m2 is not None:
            m2.close()


def test_two_runs_of_a_step_are_bit_identical_where_sums_have_a_fixed_order():
    """Losses, boundary activations, embedding gradients (sorted, not atomic, scatter) and every weight-matrix
    gradient of this size (no split contraction) are identical bit for bit between two runs; bias and LayerNorm
    parameter gradients are summed with floating-point atomics and only agree to rounding."""
    w = wl.Workload("det", K=3, Lc=1, d=128, H=2, F=256, V=64, T=128, B=6, n=2, zipf=True)   # few ids: long runs per token
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, w.B, w.T, attn_bwd="two_kernels")   # the one-sweep form sums dQ atomically
    try:
        m.set_params(P)
        runs = []
        for _ in range(2):
            m.train_step(tok, tgt)
            losses = m.get_losses()
            m.sync()
            runs.append((losses, [m.get_boundary(k, w.ntok) for k in range(w.K + 1)], {nm: m.get_grad(nm) for nm in m.names}))
        assert np.array_equal(runs[0][0], runs[1][0])
        for a, b in zip(runs[0][1], runs[1][1]):
            assert np.array_equal(a, b)
        for nm in m.names:
            a, b = runs[0][2][nm], runs[1][2][nm]
            if a.ndim == 2:
                assert np.array_equal(a, b), nm
            else:
                assert np.linalg.norm(a - b) <= 1e-5 * max(np.linalg.norm(a), 1e-30), nm
        # and the sorted scatter is right: against the oracle
        _, OG = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, 2)
        g = runs[0][2]["wte"].astype(np.float64)
        assert np.linalg.norm(g - OG["wte"]) / np.linalg.norm(OG["wte"]) < 2e-2
    finally:
        m.close()


@pytest.mark.parametrize("rule", ["sum", "far", "mean"])
@pytest.mark.parametrize("n", [1, 2, 3, 4])
def test_pipeline_placement_on_one_device_reproduces_the_single_device_step(n, rule):
    """All components mapped to device 0 but exchanged through the copy path (receive buffers owned by the
    consumer): the copies issued are exactly the planned ones, at most n-1 gradients per boundary, and the result
    equals the single-device step bit for bit wherever sums have a fixed order."""
    w = wl.Workload("k4l", K=4, Lc=1, d=128, H=2, F=256, V=500, T=64, B=2, n=n, zipf=True)
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    res = {}
    for placement in ("single", "pipeline"):
        m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, n, w.B, w.T, placement=placement, attn_bwd="two_kernels")
        try:
            m.set_params(P)
            if rule != "sum":
                m.set_rule(rule)
            m.train_step(tok, tgt, adamw=HP)
            losses = m.get_losses()
            m.sync()
            res[placement] = (losses, {nm: m.get_grad(nm) for nm in m.names}, {nm: m.get_param(nm) for nm in m.names},
                              m.last_transfers())
        finally:
            m.close()
    assert res["single"][3] == []
    plan = il.pipeline_transfers(w.K, n, rule)
    assert sorted(res["pipeline"][3]) == sorted(plan)
    for b in range(w.K - 1):
        assert sum(1 for d_, bb, _ in plan if d_ == 1 and bb == b) <= n - 1
        assert sum(1 for d_, bb, _ in plan if d_ == 0 and bb == b) == 1
    assert np.array_equal(res["single"][0], res["pipeline"][0])
    for nm, a in res["single"][1].items():
        b = res["pipeline"][1][nm]
        if a.ndim == 2:
            assert np.array_equal(a, b), nm
        else:
            assert np.linalg.norm(a - b) <= 1e-5 * max(np.linalg.norm(a), 1e-30), nm
    for nm, a in res["single"][2].items():
        assert np.max(np.abs(a - res["pipeline"][2][nm])) < 1e-6, nm


def test_noalloc_status_reports_no_error():
    assert il.op_attention_bwd_noalloc_status() == 0


_STEP_DIGEST = r"""
import hashlib, sys
import numpy as np
import workloads as wl
from paper_2010_04116_b200 import Model
w = wl.Workload("det", K=3, Lc=1, d=128, H=2, F=256, V=64, T=128, B=6, n=2, zipf=True)
P = wl.draw_params(w)
tok, tgt = wl.draw_tokens(w)
m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, 2, w.B, w.T, attn_bwd="two_kernels")
m.set_params(P)
m.train_step(tok, tgt)
losses = m.get_losses()
m.sync()
h = hashlib.sha256(np.asarray(losses, dtype=np.float32).tobytes())
for k in range(w.K + 1):
    h.update(np.ascontiguousarray(m.get_boundary(k, w.ntok)).tobytes())
for nm in m.names:
    g = m.get_grad(nm)
    if g.ndim == 2:
        h.update(np.ascontiguousarray(g).tobytes())
m.close()
print("DIGEST", h.hexdigest())
"""


def test_dependent_launch_and_ordinary_launch_give_identical_bits():
    """Kernels launched so that they may become resident while their predecessor drains (the default) wait for
    it before touching memory: losses, boundary activations and weight-matrix gradients are bit for bit those
    of the same step launched in ordinary stream order (two fresh processes; the switch is read once)."""
    import os
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    digests = []
    for off in ("0", "1"):
        env = dict(os.environ, IL_NO_DEPENDENT_LAUNCH=off, PYTHONPATH=root)
        out = subprocess.run([sys.executable, "-c", _STEP_DIGEST], cwd=root, env=env, capture_output=True, text=True,
                             timeout=600)
        assert out.returncode == 0, out.stderr[-2000:]
        digests.append([l for l in out.stdout.splitlines() if l.startswith("DIGEST")][0])
    assert digests[0] == digests[1]
