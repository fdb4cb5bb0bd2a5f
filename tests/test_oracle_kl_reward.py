"""Pins for the oracle's KL-in-reward variant: R'_b = R_b - beta * sum_t mask_t k(old_t, ref_t)."""
import math

import numpy as np

from oracle import rlf_oracle as orc
from tests.util import read_golden


def _problem(seed, B=5):
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, 40, size=B)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    old = rng.normal(-2.0, 1.0, size=T).astype(np.float32)
    ref = (old + rng.normal(0.0, 0.4, size=T)).astype(np.float32)
    mask = (rng.random(T) < 0.6).astype(np.uint8)
    r = rng.random(B).astype(np.float32)
    return r, old, ref, mask, cu


def test_hand_worked_cases():
    """tests/golden/kl_reward_cases.txt: one response, differences d = old - ref listed per token."""
    for kind, beta, reward, ds, masks, want in read_golden("kl_reward_cases.txt"):
        d = np.array([float(x) for x in ds.split()], np.float32)
        m = np.array([int(x) for x in masks.split()], np.uint8)
        ref = np.linspace(-3.0, -1.0, len(d)).astype(np.float32)
        # old = ref + d must hold exactly in fp32 for the hand values to apply: the fixture's d are dyadic
        old = (ref.astype(np.float64) + d).astype(np.float32)
        assert np.array_equal(old.astype(np.float64) - ref, d.astype(np.float64))
        out, _ = orc.kl_in_reward([float(reward)], old, ref, m, [0, len(d)], float(beta), int(kind))
        assert abs(out[0] - float(want)) < 1e-12, (kind, out[0], want)


def test_identical_policies_leave_the_reward_unchanged():
    r, old, ref, mask, cu = _problem(0)
    for kind in (0, 1, 2):
        out, kl = orc.kl_in_reward(r, old, old, mask, cu, 0.3, kind)
        assert np.array_equal(out, r.astype(np.float64)) and np.all(kl == 0.0)


def test_constant_difference_closed_forms():
    """old - ref = d on every token: the penalty is n_b k(d), n_b the number of unmasked tokens."""
    r, old, _, mask, cu = _problem(1)
    d = 0.375                                   # dyadic: old - d is exact in fp32 for these magnitudes
    old = np.round(old * 64) / 64
    ref = (old - d).astype(np.float32)
    nb = np.array([mask[cu[b]:cu[b + 1]].sum() for b in range(len(r))], np.float64)
    k = {0: d, 1: 0.5 * d * d, 2: math.exp(-d) + d - 1.0}
    for kind in (0, 1, 2):
        out, kl = orc.kl_in_reward(r, old, ref, mask, cu, 0.01, kind)
        assert np.allclose(kl, nb * k[kind], rtol=1e-13, atol=0)
        assert np.allclose(out, r - 0.01 * nb * k[kind], rtol=1e-13, atol=1e-15)


def test_against_numpy_segment_sums():
    r, old, ref, mask, cu = _problem(2, B=9)
    d = old.astype(np.float64) - ref.astype(np.float64)
    per_token = {0: d, 1: 0.5 * d * d, 2: np.expm1(-d) + d}
    for kind in (0, 1, 2):
        want = np.add.reduceat(per_token[kind] * mask, cu[:-1])
        out, kl = orc.kl_in_reward(r, old, ref, mask, cu, 0.05, kind)
        assert np.allclose(kl, want, rtol=1e-12, atol=1e-14)
        assert np.allclose(out, r - 0.05 * want, rtol=1e-12, atol=1e-14)


def test_k3_and_k2_are_nonnegative_and_k1_is_antisymmetric():
    r, old, ref, mask, cu = _problem(3)
    for kind in (1, 2):
        assert np.all(orc.kl_in_reward(r, old, ref, mask, cu, 1.0, kind)[1] >= 0.0)
    a = orc.kl_in_reward(r, old, ref, mask, cu, 1.0, 0)[1]
    b = orc.kl_in_reward(r, ref, old, mask, cu, 1.0, 0)[1]
    assert np.allclose(a, -b, atol=1e-15)
    # k3 is NOT symmetric in its arguments: exp(-d) + d - 1 differs from exp(d) - d - 1
    c = orc.kl_in_reward(r, old, ref, mask, cu, 1.0, 2)[1]
    e = orc.kl_in_reward(r, ref, old, mask, cu, 1.0, 2)[1]
    assert not np.allclose(c, e, rtol=1e-3)


def test_masked_tokens_and_other_responses_do_not_count():
    r, old, ref, mask, cu = _problem(4)
    base, _ = orc.kl_in_reward(r, old, ref, mask, cu, 0.2, 2)
    ref2 = ref.copy()
    ref2[mask == 0] += 5.0                       # perturb only masked tokens
    assert np.array_equal(orc.kl_in_reward(r, old, ref2, mask, cu, 0.2, 2)[0], base)
    # perturbing response 1 changes response 1 only
    ref3 = ref.copy()
    ref3[cu[1]:cu[2]] += 0.25
    out3, _ = orc.kl_in_reward(r, old, ref3, np.ones_like(mask), cu, 0.2, 2)
    base1, _ = orc.kl_in_reward(r, old, ref, np.ones_like(mask), cu, 0.2, 2)
    changed = out3 != base1
    assert changed[1] and not changed[[0, 2, 3, 4]].any()
    # concatenation: two batches side by side give the two results side by side
    r2, old2, refb, mask2, cu2 = _problem(5, B=3)
    both, _ = orc.kl_in_reward(np.concatenate([r, r2]), np.concatenate([old, old2]), np.concatenate([ref, refb]),
                               np.concatenate([mask, mask2]), np.concatenate([cu, cu[-1] + cu2[1:]]), 0.2, 2)
    sep2, _ = orc.kl_in_reward(r2, old2, refb, mask2, cu2, 0.2, 2)
    assert np.array_equal(both, np.concatenate([base, sep2]))


def test_beta_zero_and_bad_arguments():
    r, old, ref, mask, cu = _problem(6)
    assert np.array_equal(orc.kl_in_reward(r, old, ref, mask, cu, 0.0, 0)[0], r.astype(np.float64))
    for bad_kind in (-1, 3):
        try:
            orc.kl_in_reward(r, old, ref, mask, cu, 0.1, bad_kind)
            assert False
        except ValueError:
            pass
    try:
        orc.kl_in_reward(r, old, ref, mask, cu[::-1].copy(), 0.1, 0)
        assert False
    except ValueError:
        pass
