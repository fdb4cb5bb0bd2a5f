"""Pins for the oracle's objective variants (asymmetric clip range, sequence-mean aggregation)."""
import math

import numpy as np
import torch

from oracle import rlf_oracle as orc


def _problem(seed, T=30, V=19, B=4):
    rng = np.random.default_rng(seed)
    z = rng.normal(size=(T, V)) * 2
    ids = rng.integers(0, V, size=T).astype(np.int32)
    seq = np.sort(rng.integers(0, B, size=T)).astype(np.int32)
    adv = rng.normal(size=B).astype(np.float32)
    mask = (rng.random(T) < 0.7).astype(np.uint8)
    new = orc.grpo_loss(z, ids, seq, adv, np.zeros(T), np.zeros(T), mask, 0.2, 0.0, want_grad=False)["logp"]
    old = (new + rng.normal(0, 0.3, size=T)).astype(np.float32)
    ref = (new + rng.normal(0, 0.3, size=T)).astype(np.float32)
    return z, ids, seq, adv, old, ref, mask


def test_symmetric_token_mean_reduces_to_the_base_objective():
    z, ids, seq, adv, old, ref, mask = _problem(0)
    a = orc.grpo_loss(z, ids, seq, adv, old, ref, mask, 0.2, 0.05)
    b = orc.grpo_loss_obj(z, ids, seq, adv, old, ref, mask, 0.2, 0.2, 0.05, aggregation=0)
    assert np.allclose(a["loss"], b["loss"], atol=1e-15) and np.allclose(a["grad"], b["grad"], atol=1e-17)
    c = orc.grpo_loss_obj(z, ids, seq, adv, old, ref, mask, 0.2, 0.2, 0.05, aggregation=0, denom=77)
    d = orc.grpo_loss(z, ids, seq, adv, old, ref, mask, 0.2, 0.05, denom=77)
    assert np.allclose(c["loss"], d["loss"], atol=1e-15)


def test_asymmetric_clip_hand_cases():
    """eps_low 0.2, eps_high 0.28: rho = 1.25, A = 1 is inside the range (pg = -1.25, gradient -1.25);
    with the symmetric 0.2 it is clipped (pg = -1.2, gradient 0).  rho = 0.75, A = -1: clipped at 0.8."""
    logp = -math.log(2.0)

    def one(A, rho, lo, hi):
        r = orc.grpo_loss_obj(np.zeros((1, 2)), [0], [0], [A], [logp - math.log(rho)], [logp], [1], lo, hi, 0.0,
                              want_coef=True)
        return r["loss"][1], -r["coef"][0], r["loss"][3]
    pg, dpg, cl = one(1.0, 1.25, 0.2, 0.28)
    assert abs(pg + 1.25) < 1e-6 and abs(dpg + 1.25) < 1e-6 and cl == 0
    pg, dpg, cl = one(1.0, 1.25, 0.2, 0.2)
    assert abs(pg + 1.2) < 1e-6 and dpg == 0 and cl == 1
    pg, dpg, cl = one(-1.0, 0.75, 0.2, 0.28)
    assert abs(pg - 0.8) < 1e-6 and dpg == 0 and cl == 1
    pg, dpg, cl = one(-1.0, 1.25, 0.2, 0.28)          # negative advantage is never clipped from above
    assert abs(pg - 1.25) < 1e-6 and abs(dpg - 1.25) < 1e-6 and cl == 0


def test_sequence_mean_closed_form_and_difference_from_token_mean():
    """Two sequences of 1 and 3 live tokens with per-token losses l: seq mean = (l0 + (l1+l2+l3)/3) / 2."""
    V = 4
    z = np.zeros((5, V))
    logp = -math.log(V)
    A = np.array([1.0, -2.0], np.float32)
    seq = np.array([0, 1, 1, 1, 1], np.int32)
    mask = np.array([1, 1, 1, 1, 0], np.uint8)
    old = np.full(5, logp, np.float32)
    r = orc.grpo_loss_obj(z, [0] * 5, seq, A, old, old, mask, 0.2, 0.2, 0.0, aggregation=1, want_coef=True)
    rho = math.exp(logp - float(old[0]))
    want = (-(rho * 1.0) + (3 * (rho * 2.0)) / 3) / 2
    assert abs(r["loss"][0] - want) < 1e-12
    tok = orc.grpo_loss_obj(z, [0] * 5, seq, A, old, old, mask, 0.2, 0.2, 0.0, aggregation=0)
    assert abs(tok["loss"][0] - (-(rho) + 3 * 2 * rho) / 4) < 1e-12
    # weights: 1/(1*2) for the lone token, 1/(3*2) for the others, 0 for the masked one
    g = -r["coef"] / np.array([-rho, 2 * rho, 2 * rho, 2 * rho, 1.0])
    assert np.allclose(g[:4], [0.5, 1 / 6, 1 / 6, 1 / 6], atol=1e-9) and r["coef"][4] == 0
    # explicit number of sequences (micro-batching): weights scale by 2 / 5
    r5 = orc.grpo_loss_obj(z, [0] * 5, seq, A, old, old, mask, 0.2, 0.2, 0.0, aggregation=1, denom=5)
    assert abs(r5["loss"][0] - want * 2 / 5) < 1e-12


def test_variants_match_torch_autograd():
    for seed, lo, hi, agg in ((1, 0.2, 0.28, 0), (2, 0.1, 0.3, 1), (3, 0.2, 0.2, 1)):
        z, ids, seq, adv, old, ref, mask = _problem(seed)
        beta = 0.07
        r = orc.grpo_loss_obj(z, ids, seq, adv, old, ref, mask, lo, hi, beta, aggregation=agg)
        zt = torch.tensor(z, requires_grad=True)
        lp = torch.log_softmax(zt, -1).gather(1, torch.tensor(ids, dtype=torch.int64)[:, None])[:, 0]
        sq = torch.tensor(seq, dtype=torch.int64)
        A = torch.tensor(adv, dtype=torch.float64)[sq]
        rho = torch.exp(lp - torch.tensor(old, dtype=torch.float64))
        pg = -torch.minimum(rho * A, torch.clamp(rho, 1 - lo, 1 + hi) * A)
        d = torch.tensor(ref, dtype=torch.float64) - lp
        ell = pg + beta * (torch.exp(d) - d - 1)
        m = torch.tensor(mask, dtype=torch.float64)
        if agg == 0:
            L = (m * ell).sum() / m.sum()
        else:
            nb = torch.zeros(len(adv), dtype=torch.float64).index_add(0, sq, m)
            per = torch.zeros(len(adv), dtype=torch.float64).index_add(0, sq, m * ell) / nb.clamp(min=1)
            L = per[nb > 0].mean()
        L.backward()
        assert abs(r["loss"][0] - L.item()) < 1e-13
        assert np.abs(r["grad"] - zt.grad.numpy()).max() < 1e-14
