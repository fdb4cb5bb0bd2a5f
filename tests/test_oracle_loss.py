"""Pins for the oracle's log-prob / clipped-ratio / k3-KL loss and its gradient.

The paper names the algorithms (Sec. 2.3) and fixes that observation tokens are excluded
(Sec. 2.2); the formulas are the textbook ones.  Pins used: closed forms of log-sum-exp, hand-worked
token cases (tests/golden/token_loss_cases.txt), identities that hold for any input, central finite
differences, and fp64 torch.log_softmax / torch.autograd as an independent library evaluation."""
import math

import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from util import read_golden


def _one_row(z, y, A=0.0, old=None, ref=None, beta=0.0, mask=1, denom=None):
    z = np.asarray(z, np.float64)[None, :]
    r = orc.grpo_loss(z, [y], [0], [A], [0.0 if old is None else old], [0.0 if ref is None else ref],
                      [mask], 0.2, beta, denom=denom, want_coef=True)
    return r


def test_constant_logits_logsumexp_is_log_V():
    for V in (1, 2, 7, 1024, 151936):
        for c in (-3.5, 0.0, 11.0, -1e30, 1e30):   # huge constants must not absorb log V
            r = _one_row(np.full(V, c), V // 2)
            assert abs(r["logp"][0] + math.log(V)) < 1e-12


def test_shift_invariance_and_dominant_logit():
    rng = np.random.default_rng(0)
    z = rng.normal(0, 3, size=300)
    a = _one_row(z, 17)["logp"][0]
    b = _one_row(z + 123.25, 17)["logp"][0]
    assert abs(a - b) < 1e-10
    z2 = np.zeros(50)
    z2[3] = 80.0
    assert abs(_one_row(z2, 3)["logp"][0]) < 1e-30 + 50 * math.exp(-80)
    assert abs(_one_row(z2, 4)["logp"][0] + 80.0) < 1e-10


def test_two_valued_row_closed_form():
    """k entries equal a, V-k equal b: lse = log(k e^a + (V-k) e^b)."""
    V, k, a, b = 1000, 37, 2.5, -1.25
    z = np.full(V, b)
    z[:k] = a
    lse = math.log(k * math.exp(a) + (V - k) * math.exp(b))
    assert abs(_one_row(z, 0)["logp"][0] - (a - lse)) < 1e-12
    assert abs(_one_row(z, V - 1)["logp"][0] - (b - lse)) < 1e-12


def test_large_magnitude_logits_do_not_overflow():
    z = np.array([1000.0, 999.0, -1000.0])
    want = -math.log1p(math.exp(-1.0))
    assert abs(_one_row(z, 0)["logp"][0] - want) < 1e-12


@pytest.mark.parametrize("dtype", ["bf16", "f32", "f64"])
def test_logp_matches_torch_log_softmax_fp64(dtype):
    g = torch.Generator().manual_seed(1)
    T, V = 9, 301
    z = torch.randn(T, V, generator=g) * 3
    ids = torch.randint(0, V, (T,), generator=g)
    if dtype == "bf16":
        zt = z.to(torch.bfloat16)
        arr = zt.view(torch.int16).numpy().view(np.uint16)
    elif dtype == "f32":
        zt = z
        arr = zt.numpy()
    else:
        zt = z.double()
        arr = zt.numpy()
    want = torch.log_softmax(zt.double(), -1).gather(1, ids[:, None])[:, 0].numpy()
    r = orc.grpo_loss(arr, ids.numpy(), np.zeros(T, np.int32), [0.0], np.zeros(T), np.zeros(T),
                      np.ones(T, np.uint8), 0.2, 0.0, want_grad=False)
    assert np.allclose(r["logp"], want, rtol=0, atol=1e-12)


def test_strided_rows():
    rng = np.random.default_rng(2)
    big = rng.normal(size=(5, 40))
    view = big[:, :33]
    ids = np.array([0, 32, 5, 7, 9], np.int32)
    a = orc.grpo_loss(view, ids, np.zeros(5, np.int32), [0.5], np.zeros(5), np.zeros(5), np.ones(5, np.uint8), 0.2, 0.1)
    b = orc.grpo_loss(np.ascontiguousarray(view), ids, np.zeros(5, np.int32), [0.5], np.zeros(5), np.zeros(5),
                      np.ones(5, np.uint8), 0.2, 0.1)
    assert np.array_equal(a["logp"], b["logp"]) and np.array_equal(a["grad"], b["grad"])


_CASES = read_golden("token_loss_cases.txt")


@pytest.mark.parametrize("row", [r for r in _CASES if r[0] != "KL"])
def test_hand_cases_clipped_surrogate(row):
    A, rho, pg, dpg, clipped = (float(x) for x in row)
    logp = -math.log(2.0)                       # two equal logits
    old = logp - math.log(rho)
    r = _one_row([0.0, 0.0], 1, A=A, old=old, ref=logp, beta=0.0)
    assert abs(r["logp"][0] - logp) < 1e-15
    assert abs(r["loss"][1] - pg) < 1e-6 and abs(r["loss"][0] - pg) < 1e-6
    assert r["loss"][3] == clipped
    assert abs(r["coef"][0] + dpg) < 1e-6
    # grad = dL/dlogp * (onehot - p), p = (1/2, 1/2)
    assert np.allclose(r["grad"][0], [-0.5 * dpg, 0.5 * dpg], atol=1e-6)


@pytest.mark.parametrize("row", [r for r in _CASES if r[0] == "KL"])
def test_hand_cases_k3(row):
    ed, kl, dkl = (float(x) for x in row[1:])
    logp = -math.log(2.0)
    ref = logp + math.log(ed)
    r = _one_row([0.0, 0.0], 0, A=0.0, old=logp, ref=ref, beta=1.0)
    assert abs(r["loss"][2] - kl) < 1e-6 and abs(r["loss"][0] - kl) < 1e-6
    assert abs(r["coef"][0] + dkl) < 1e-6
    assert r["loss"][2] >= 0.0


def _random_problem(rng, T=12, V=23, B=3, dtype=np.float64, scale=2.0):
    z = (rng.normal(size=(T, V)) * scale).astype(dtype)
    ids = rng.integers(0, V, size=T).astype(np.int32)
    seq = np.sort(rng.integers(0, B, size=T)).astype(np.int32)
    adv = rng.normal(size=B).astype(np.float32)
    mask = (rng.random(T) < 0.7).astype(np.uint8)
    new = orc.grpo_loss(z, ids, seq, adv, np.zeros(T), np.zeros(T), mask, 0.2, 0.0, want_grad=False)["logp"]
    old = (new + rng.normal(0, 0.3, size=T)).astype(np.float32)
    ref = (new + rng.normal(0, 0.3, size=T)).astype(np.float32)
    return z, ids, seq, adv, old, ref, mask, new


def test_loss_is_minus_masked_mean_advantage_when_old_equals_new():
    rng = np.random.default_rng(3)
    z, ids, seq, adv, old, ref, mask, new = _random_problem(rng, T=64, V=50)
    # fp32 storage of old_logp rounds it; use logits for which logp is exactly representable:
    # constant rows give logp = -log V; pick V = 64 and scale so that fp32(-log 64) error is ~1e-7
    new32 = new.astype(np.float32)
    r = orc.grpo_loss(z, ids, seq, adv, new32, new32, mask, 0.2, 0.0)
    want = -(adv.astype(np.float64)[seq] * mask).sum() / mask.sum()
    assert abs(r["loss"][0] - want) < 1e-6
    assert r["loss"][3] == 0.0
    # with beta > 0 and ref = new the KL term vanishes (to fp32 rounding of ref, squared)
    r2 = orc.grpo_loss(z, ids, seq, adv, new32, new32, mask, 0.2, 0.7)
    assert r2["loss"][2] < 1e-12 and abs(r2["loss"][0] - want) < 1e-6


def test_kl_zero_and_gradient_zero_when_ref_equals_new_exactly():
    """Constant rows over V = 2^k logits have logp = -k log 2; choose values whose fp32 rounding
    is taken on both sides so ref == logp to the last bit is not needed: d is ~1e-8, kl ~ d^2/2."""
    z = np.zeros((4, 16))
    logp = -math.log(16.0)
    ref = np.full(4, logp, np.float32)
    r = orc.grpo_loss(z, [0, 1, 2, 3], [0] * 4, [0.0], ref, ref, [1] * 4, 0.2, 1.0, want_coef=True)
    d = float(ref[0]) - logp
    assert abs(r["loss"][2] - (math.exp(d) - d - 1)) < 1e-18
    assert r["loss"][2] < 1e-14 and np.abs(r["coef"]).max() < 1e-7


def test_gradient_rows_sum_to_zero_and_masked_rows_are_zero():
    rng = np.random.default_rng(4)
    z, ids, seq, adv, old, ref, mask, new = _random_problem(rng, T=40, V=37)
    r = orc.grpo_loss(z, ids, seq, adv, old, ref, mask, 0.2, 0.05, want_coef=True)
    g = r["grad"]
    assert np.abs(g.sum(axis=1)).max() < 1e-15
    assert (g[mask == 0] == 0).all() and np.abs(g[mask == 1]).max() > 0
    # target column: coef * (p_y - 1); any other column: coef * p_v
    p = np.exp(z - np.log(np.exp(z).sum(1, keepdims=True)))
    want = r["coef"][:, None] * (p - np.eye(z.shape[1])[ids])
    assert np.allclose(g, want, atol=1e-15)


def test_gradient_matches_central_finite_differences():
    rng = np.random.default_rng(5)
    T, V = 8, 16
    z, ids, seq, adv, old, ref, mask, new = _random_problem(rng, T=T, V=V)
    beta = 0.3
    r = orc.grpo_loss(z, ids, seq, adv, old, ref, mask, 0.2, beta)
    h = 1e-6
    fd = np.zeros_like(z)
    for t in range(T):
        for v in range(V):
            zp = z.copy(); zp[t, v] += h
            zm = z.copy(); zm[t, v] -= h
            lp = orc.grpo_loss(zp, ids, seq, adv, old, ref, mask, 0.2, beta, want_grad=False)["loss"][0]
            lm = orc.grpo_loss(zm, ids, seq, adv, old, ref, mask, 0.2, beta, want_grad=False)["loss"][0]
            fd[t, v] = (lp - lm) / (2 * h)
    assert np.abs(fd - r["grad"]).max() < 1e-8
    assert np.abs(r["grad"]).max() > 1e-3


def _torch_loss(z, ids, seq, adv, old, ref, mask, eps, beta, denom=None):
    """The same objective written with library ops, for autograd."""
    logp = torch.log_softmax(z, -1).gather(1, ids[:, None])[:, 0]
    A = adv[seq]
    rho = torch.exp(logp - old)
    pg = -torch.minimum(rho * A, torch.clamp(rho, 1 - eps, 1 + eps) * A)
    d = ref - logp
    kl = torch.exp(d) - d - 1
    n = mask.sum() if denom is None else torch.tensor(float(denom), dtype=z.dtype)
    n = torch.clamp(n, min=1.0)
    return (mask * (pg + beta * kl)).sum() / n, (mask * pg).sum() / n, (mask * kl).sum() / n


@pytest.mark.parametrize("seed,denom", [(6, None), (7, 1000), (8, None)])
def test_loss_and_gradient_match_torch_autograd_fp64(seed, denom):
    rng = np.random.default_rng(seed)
    z, ids, seq, adv, old, ref, mask, new = _random_problem(rng, T=30, V=41, B=4)
    r = orc.grpo_loss(z, ids, seq, adv, old, ref, mask, 0.2, 0.04, denom=denom)
    zt = torch.tensor(z, requires_grad=True)
    L, PG, KL = _torch_loss(zt, torch.tensor(ids, dtype=torch.int64), torch.tensor(seq, dtype=torch.int64),
                            torch.tensor(adv, dtype=torch.float64), torch.tensor(old, dtype=torch.float64),
                            torch.tensor(ref, dtype=torch.float64), torch.tensor(mask, dtype=torch.float64),
                            0.2, 0.04, denom)
    L.backward()
    assert abs(r["loss"][0] - L.item()) < 1e-13
    assert abs(r["loss"][1] - PG.item()) < 1e-13 and abs(r["loss"][2] - KL.item()) < 1e-13
    assert np.abs(r["grad"] - zt.grad.numpy()).max() < 1e-14
    # the clip fraction is genuinely exercised by this input
    assert 0.0 < r["loss"][3] < 1.0


def test_micro_batches_with_global_denominator_add_up():
    rng = np.random.default_rng(9)
    z, ids, seq, adv, old, ref, mask, new = _random_problem(rng, T=24, V=19)
    full = orc.grpo_loss(z, ids, seq, adv, old, ref, mask, 0.2, 0.1)
    N = int(mask.sum())
    parts = [orc.grpo_loss(z[a:b], ids[a:b], seq[a:b], adv, old[a:b], ref[a:b], mask[a:b], 0.2, 0.1, denom=N)
             for a, b in ((0, 8), (8, 16), (16, 24))]
    assert abs(sum(p["loss"][0] for p in parts) - full["loss"][0]) < 1e-14
    assert np.allclose(np.concatenate([p["grad"] for p in parts]), full["grad"], atol=1e-16)


def test_all_masked_batch_gives_zero_loss_and_gradient():
    rng = np.random.default_rng(10)
    z, ids, seq, adv, old, ref, mask, new = _random_problem(rng, T=6, V=9)
    r = orc.grpo_loss(z, ids, seq, adv, old, ref, np.zeros(6, np.uint8), 0.2, 0.1)
    assert (r["loss"] == 0).all() and (r["grad"] == 0).all() and np.isfinite(r["logp"]).all()


def test_out_of_range_target_is_an_error():
    with pytest.raises(ValueError):
        _one_row([0.0, 1.0], 2)
