"""Pins for the oracle's fused LM-head variant: logits are the contraction H W^T (the policy head
behind pi_theta of Sec. 2.2), the loss is the same, gradients follow by the chain rule."""
import numpy as np
import torch

from oracle import rlf_oracle as orc


def _bf16(x):
    t = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16), t.double().numpy()


def _problem(seed, T=10, D=12, V=17, B=3):
    rng = np.random.default_rng(seed)
    Hb, H = _bf16(rng.normal(size=(T, D)))
    Wb, W = _bf16(rng.normal(size=(V, D)) * 0.5)
    ids = rng.integers(0, V, size=T).astype(np.int32)
    seq = np.sort(rng.integers(0, B, size=T)).astype(np.int32)
    adv = rng.normal(size=B).astype(np.float32)
    mask = (rng.random(T) < 0.7).astype(np.uint8)
    z = H @ W.T
    new = orc.grpo_loss(z, ids, seq, adv, np.zeros(T), np.zeros(T), mask, 0.2, 0.0, want_grad=False)["logp"]
    old = (new + rng.normal(0, 0.3, size=T)).astype(np.float32)
    ref = (new + rng.normal(0, 0.3, size=T)).astype(np.float32)
    return Hb, H, Wb, W, ids, seq, adv, old, ref, mask


def test_logits_are_the_fp64_contraction_with_untransposed_layouts():
    Hb, H, Wb, W, ids, seq, adv, old, ref, mask = _problem(0)
    r = orc.fused_lmhead_grpo(Hb, Wb, ids, seq, adv, old, ref, mask, 0.2, 0.1, want_z=True)
    assert np.abs(r["z"] - H @ W.T).max() < 1e-13          # numpy matmul: library contraction
    same = orc.grpo_loss(H @ W.T, ids, seq, adv, old, ref, mask, 0.2, 0.1)
    assert np.allclose(r["logp"], same["logp"], atol=1e-13) and np.allclose(r["loss"], same["loss"], atol=1e-13)
    assert np.allclose(r["grad_hidden"], same["grad"] @ W, atol=1e-14)
    assert np.allclose(r["grad_W"], same["grad"].T @ H, atol=1e-14)


def test_gradients_match_torch_autograd_fp64():
    Hb, H, Wb, W, ids, seq, adv, old, ref, mask = _problem(1)
    r = orc.fused_lmhead_grpo(Hb, Wb, ids, seq, adv, old, ref, mask, 0.2, 0.05)
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    z = Ht @ Wt.t()
    logp = torch.log_softmax(z, -1).gather(1, torch.tensor(ids, dtype=torch.int64)[:, None])[:, 0]
    A = torch.tensor(adv, dtype=torch.float64)[torch.tensor(seq, dtype=torch.int64)]
    rho = torch.exp(logp - torch.tensor(old, dtype=torch.float64))
    pg = -torch.minimum(rho * A, torch.clamp(rho, 0.8, 1.2) * A)
    d = torch.tensor(ref, dtype=torch.float64) - logp
    m = torch.tensor(mask, dtype=torch.float64)
    L = (m * (pg + 0.05 * (torch.exp(d) - d - 1))).sum() / m.sum()
    L.backward()
    assert abs(r["loss"][0] - L.item()) < 1e-13
    assert np.abs(r["grad_hidden"] - Ht.grad.numpy()).max() < 1e-14
    assert np.abs(r["grad_W"] - Wt.grad.numpy()).max() < 1e-14


def test_invariants_of_the_head_gradients():
    Hb, H, Wb, W, ids, seq, adv, old, ref, mask = _problem(2, T=14, D=9, V=21)
    r = orc.fused_lmhead_grpo(Hb, Wb, ids, seq, adv, old, ref, mask, 0.2, 0.05)
    # every row of grad_z sums to zero, so the columns of grad_W sum to zero over the vocabulary
    assert np.abs(r["grad_W"].sum(axis=0)).max() < 1e-14
    assert (r["grad_hidden"][mask == 0] == 0).all()
    # grad_hidden[t] = coef_t (E_p[W] - W_y)
    z = H @ W.T
    g = orc.grpo_loss(z, ids, seq, adv, old, ref, mask, 0.2, 0.05, want_coef=True)
    p = np.exp(z - z.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    want = g["coef"][:, None] * (p @ W - W[ids])
    assert np.allclose(r["grad_hidden"], want, atol=1e-14)


def test_finite_differences_through_the_head():
    """bf16 inputs cannot be perturbed by 1e-6, so the check differentiates the fp64 logits path
    composed with the contraction: dL/dH[t,k] ~ (L(H + h e_tk) - L(H - h e_tk)) / 2h."""
    Hb, H, Wb, W, ids, seq, adv, old, ref, mask = _problem(3, T=5, D=4, V=7)
    r = orc.fused_lmhead_grpo(Hb, Wb, ids, seq, adv, old, ref, mask, 0.2, 0.2)

    def L(Hx, Wx):
        return orc.grpo_loss(Hx @ Wx.T, ids, seq, adv, old, ref, mask, 0.2, 0.2, want_grad=False)["loss"][0]
    h = 1e-6
    for (t, k) in [(0, 0), (1, 3), (4, 2), (2, 1)]:
        Hp, Hm = H.copy(), H.copy()
        Hp[t, k] += h; Hm[t, k] -= h
        assert abs((L(Hp, W) - L(Hm, W)) / (2 * h) - r["grad_hidden"][t, k]) < 1e-8
    for (v, k) in [(0, 0), (6, 3), (3, 1), (int(ids[0]), 2)]:
        Wp, Wm = W.copy(), W.copy()
        Wp[v, k] += h; Wm[v, k] -= h
        assert abs((L(H, Wp) - L(H, Wm)) / (2 * h) - r["grad_W"][v, k]) < 1e-8


def test_objective_variant_of_the_head_reduces_and_composes():
    Hb, H, Wb, W, ids, seq, adv, old, ref, mask = _problem(4)
    base = orc.fused_lmhead_grpo(Hb, Wb, ids, seq, adv, old, ref, mask, 0.2, 0.05)
    same = orc.fused_lmhead_grpo_obj(Hb, Wb, ids, seq, adv, old, ref, mask, 0.2, 0.2, 0.05, aggregation=0)
    for k in ("logp", "loss", "grad_hidden", "grad_W"):
        assert np.allclose(base[k], same[k], atol=1e-15), k
    # composition with the logits-path variant on the fp64 contraction (numpy matmul as the library step)
    for agg in (0, 1):
        r = orc.fused_lmhead_grpo_obj(Hb, Wb, ids, seq, adv, old, ref, mask, 0.1, 0.3, 0.05, aggregation=agg)
        g = orc.grpo_loss_obj(H @ W.T, ids, seq, adv, old, ref, mask, 0.1, 0.3, 0.05, aggregation=agg)
        assert np.allclose(r["loss"], g["loss"], atol=1e-13) and np.allclose(r["logp"], g["logp"], atol=1e-13)
        assert np.allclose(r["grad_hidden"], g["grad"] @ W, atol=1e-14)
        assert np.allclose(r["grad_W"], g["grad"].T @ H, atol=1e-14)


def test_objective_variant_of_the_head_matches_torch_autograd_fp64():
    """Asymmetric clip range with the sequence mean: L = (1/S) sum_b (1/n_b) sum_{t in b} mask_t l_t."""
    Hb, H, Wb, W, ids, seq, adv, old, ref, mask = _problem(5, T=16, B=4)
    lo, hi, beta = 0.15, 0.4, 0.07
    r = orc.fused_lmhead_grpo_obj(Hb, Wb, ids, seq, adv, old, ref, mask, lo, hi, beta, aggregation=1)
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    logp = torch.log_softmax(Ht @ Wt.t(), -1).gather(1, torch.tensor(ids, dtype=torch.int64)[:, None])[:, 0]
    seq_t = torch.tensor(seq, dtype=torch.int64)
    A = torch.tensor(adv, dtype=torch.float64)[seq_t]
    rho = torch.exp(logp - torch.tensor(old, dtype=torch.float64))
    pg = -torch.minimum(rho * A, torch.clamp(rho, 1 - lo, 1 + hi) * A)
    d = torch.tensor(ref, dtype=torch.float64) - logp
    m = torch.tensor(mask, dtype=torch.float64)
    tok = m * (pg + beta * (torch.exp(d) - d - 1))
    L = 0.0
    S = 0
    for b in range(4):
        sel = seq_t == b
        if m[sel].sum() > 0:
            L = L + tok[sel].sum() / m[sel].sum()
            S += 1
    L = L / S
    L.backward()
    assert abs(r["loss"][0] - L.item()) < 1e-13
    assert np.abs(r["grad_hidden"] - Ht.grad.numpy()).max() < 1e-14
    assert np.abs(r["grad_W"] - Wt.grad.numpy()).max() < 1e-14


def test_forward_only_head_log_prob_and_entropy():
    import math
    Hb, H, Wb, W, ids, seq, adv, old, ref, mask = _problem(6, T=9, D=6, V=13)
    logp, ent = orc.fused_lmhead_logp_entropy(Hb, Wb, ids)
    # composition with the logits-path function on numpy's fp64 contraction
    lp2, ent2 = orc.logp_entropy(H @ W.T, ids)
    assert np.allclose(logp, lp2, atol=1e-13) and np.allclose(ent, ent2, atol=1e-13)
    # fp64 torch
    z = torch.tensor(H) @ torch.tensor(W).t()
    ls = torch.log_softmax(z, -1)
    assert np.allclose(logp, ls.gather(1, torch.tensor(ids, dtype=torch.int64)[:, None])[:, 0].numpy(), atol=1e-13)
    assert np.allclose(ent, -(ls.exp() * ls).sum(-1).numpy(), atol=1e-13)
    # a zero head gives the uniform distribution: log-prob -ln V, entropy ln V, whatever the hidden states
    Zb, _ = _bf16(np.zeros((13, 6)))
    logp0, ent0 = orc.fused_lmhead_logp_entropy(Hb, Zb, ids)
    assert np.allclose(logp0, -math.log(13), atol=1e-15) and np.allclose(ent0, math.log(13), atol=1e-15)
    # agreement with the training path's log-prob
    r = orc.fused_lmhead_grpo(Hb, Wb, ids, seq, adv, old, ref, mask, 0.2, 0.05, want_grad_hidden=False, want_grad_W=False)
    assert np.allclose(r["logp"], logp, atol=1e-13)
    assert orc.fused_lmhead_logp_entropy(Hb, Wb, ids, want_entropy=False)[1] is None
