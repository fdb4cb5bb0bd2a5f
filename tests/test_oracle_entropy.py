"""Pins for the oracle's forward-only log-prob / entropy (policy softmax of Sec. 2.2; the pass that
yields old_logp / ref_logp for the update of Sec. 2.3.1)."""
import math

import numpy as np
import torch

from oracle import rlf_oracle as orc


def test_uniform_row_has_entropy_log_V_and_logp_minus_log_V():
    for V in (1, 2, 17, 4096):
        lp, h = orc.logp_entropy(np.full((1, V), 2.5), [V - 1])
        assert abs(lp[0] + math.log(V)) < 1e-12 and abs(h[0] - math.log(V)) < 1e-12


def test_two_point_distribution_closed_form():
    """logits (a, b): p = sigmoid(a - b); H = -p ln p - (1-p) ln(1-p)."""
    a, b = 1.25, -0.5
    p = 1 / (1 + math.exp(b - a))
    lp, h = orc.logp_entropy(np.array([[a, b]]), [0])
    assert abs(lp[0] - math.log(p)) < 1e-14
    assert abs(h[0] + p * math.log(p) + (1 - p) * math.log(1 - p)) < 1e-14


def test_dominant_and_minus_infinity_entries():
    z = np.zeros((2, 8))
    z[0, 3] = 200.0                       # one-hot in the limit: entropy -> 0
    z[1, ::2] = -np.inf                   # four entries of probability exactly zero: H = ln 4
    lp, h = orc.logp_entropy(z, [3, 1])
    assert abs(lp[0]) < 1e-80 and h[0] < 1e-80
    assert abs(h[1] - math.log(4)) < 1e-14 and abs(lp[1] + math.log(4)) < 1e-14


def test_matches_torch_fp64_and_shift_invariance():
    g = torch.Generator().manual_seed(3)
    z = torch.randn(7, 301, generator=g, dtype=torch.float64) * 3
    ids = torch.randint(0, 301, (7,), generator=g)
    ls = torch.log_softmax(z, -1)
    want_h = -(ls.exp() * ls).sum(-1).numpy()
    want_lp = ls.gather(1, ids[:, None])[:, 0].numpy()
    lp, h = orc.logp_entropy(z.numpy(), ids.numpy())
    assert np.allclose(lp, want_lp, atol=1e-12) and np.allclose(h, want_h, atol=1e-12)
    lp2, h2 = orc.logp_entropy((z + 1e3).numpy(), ids.numpy())
    assert np.allclose(lp2, lp, atol=1e-9) and np.allclose(h2, h, atol=1e-9)


def test_agrees_with_the_loss_path_logp_and_bf16_input():
    rng = np.random.default_rng(5)
    zt = torch.tensor(rng.normal(size=(5, 64)) * 2, dtype=torch.float32).to(torch.bfloat16)
    arr = zt.view(torch.int16).numpy().view(np.uint16)
    ids = rng.integers(0, 64, size=5).astype(np.int32)
    lp, h = orc.logp_entropy(arr, ids)
    r = orc.grpo_loss(arr, ids, np.zeros(5, np.int32), [0.0], np.zeros(5), np.zeros(5), np.ones(5, np.uint8), 0.2, 0.0,
                      want_grad=False)
    assert np.array_equal(lp, r["logp"])
    assert (h > 0).all() and (h <= math.log(64) + 1e-12).all()
