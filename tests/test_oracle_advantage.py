"""Pins for the oracle's group-relative advantage (GRPO is named in Sec. 2.3.2 / Fig. 4 without a
formula; the definition is (r - mean_group) / (std_group + eps))."""
import numpy as np

from oracle import rlf_oracle as orc


def test_zero_mean_unit_std_per_group():
    rng = np.random.default_rng(0)
    G, P = 8, 5
    r = rng.random(G * P).astype(np.float32)
    for unbiased in (True, False):
        a = orc.group_advantage(r, group_size=G, eps=0.0, unbiased=unbiased).reshape(P, G)
        assert np.allclose(a.mean(axis=1), 0.0, atol=1e-12)
        assert np.allclose(a.std(axis=1, ddof=1 if unbiased else 0), 1.0, atol=1e-12)


def test_closed_form_two_member_group():
    """r = (0, 1): mean 1/2; unbiased std = sqrt(1/2) -> A = -+1/sqrt(2); biased std = 1/2 -> A = -+1."""
    r = np.array([0.0, 1.0], np.float32)
    a = orc.group_advantage(r, group_size=2, eps=0.0, unbiased=True)
    assert np.allclose(a, [-1 / np.sqrt(2), 1 / np.sqrt(2)], atol=1e-15)
    a = orc.group_advantage(r, group_size=2, eps=0.0, unbiased=False)
    assert np.allclose(a, [-1.0, 1.0], atol=1e-15)


def test_closed_form_with_eps():
    """r = (1, 3, 5): mean 3, unbiased std 2 -> A = (-2, 0, 2) / (2 + eps)."""
    r = np.array([1.0, 3.0, 5.0], np.float32)
    a = orc.group_advantage(r, group_size=3, eps=0.5, unbiased=True)
    assert np.allclose(a, np.array([-2.0, 0.0, 2.0]) / 2.5, atol=1e-15)


def test_library_cross_check_against_numpy_std():
    rng = np.random.default_rng(3)
    r = rng.normal(size=24).astype(np.float32)
    a = orc.group_advantage(r, group_size=6, eps=1e-6, unbiased=True).reshape(4, 6)
    r64 = r.astype(np.float64).reshape(4, 6)
    want = (r64 - r64.mean(1, keepdims=True)) / (np.std(r64, axis=1, ddof=1, keepdims=True) + 1e-6)
    assert np.allclose(a, want, rtol=1e-13, atol=1e-13)


def test_affine_invariance_and_permutation_equivariance():
    rng = np.random.default_rng(4)
    r = rng.random(16).astype(np.float64)
    r32 = r.astype(np.float32)
    a = orc.group_advantage(r32, group_size=8, eps=0.0)
    # power-of-two scale and an offset exactly representable keep float32 inputs exact
    a2 = orc.group_advantage((r32 * 4.0 + 2.0).astype(np.float32), group_size=8, eps=0.0)
    assert np.allclose(a, a2, atol=1e-5)
    perm = np.concatenate([rng.permutation(8), 8 + rng.permutation(8)])
    ap = orc.group_advantage(r32[perm], group_size=8, eps=0.0)
    assert np.allclose(ap, a[perm], atol=1e-12)


def test_degenerate_groups_give_zero():
    r = np.array([1, 1, 1, 1, 0, 1, 0, 1], np.float32)
    a = orc.group_advantage(r, group_size=4, eps=1e-6)
    assert (a[:4] == 0.0).all() and abs(a[4:].sum()) < 1e-12 and a[5] > 0
    a1 = orc.group_advantage(np.array([0.3, 0.9], np.float32), group_size=1, eps=1e-6)
    assert (a1 == 0.0).all()


def test_degenerate_groups_give_zero_also_without_eps():
    # eps = 0: the formula reads 0 / 0 for a group without spread; the reading is A = 0 (no signal),
    # never NaN, for both std conventions, for a single-member group, and beside a healthy group
    r = np.array([1, 1, 1, 1, 0, 1, 0, 1], np.float32)
    for unbiased in (True, False):
        a = orc.group_advantage(r, group_size=4, eps=0.0, unbiased=unbiased)
        assert np.isfinite(a).all() and (a[:4] == 0.0).all()
        sd = np.std(r[4:].astype(np.float64), ddof=1 if unbiased else 0)
        assert np.allclose(a[4:], (r[4:] - 0.5) / sd, atol=1e-12)
    a1 = orc.group_advantage(np.array([0.3, 0.9], np.float32), group_size=1, eps=0.0)
    assert (a1 == 0.0).all()


def test_explicit_group_ids_match_contiguous_groups():
    rng = np.random.default_rng(5)
    r = rng.random(12).astype(np.float32)
    a = orc.group_advantage(r, group_size=4)
    gid = np.repeat(np.arange(3), 4).astype(np.int32)
    perm = rng.permutation(12)
    ap = orc.group_advantage(r[perm], group_id=gid[perm], num_groups=3)
    assert np.allclose(ap, a[perm], atol=1e-12)


def test_ragged_last_group():
    r = np.array([0.0, 1.0, 2.0, 5.0, 7.0], np.float32)
    a = orc.group_advantage(r, group_size=3, eps=0.0)
    assert np.allclose(a[:3], [-1.0, 0.0, 1.0]) and np.allclose(a[3:], [-1 / np.sqrt(2), 1 / np.sqrt(2)])


def test_rule_reward_eq1():
    """Eq. 1: R = sum_i w_i r_i."""
    s = np.array([[1.0, 0.0, 0.5], [0.0, 1.0, 1.0]], np.float32)
    w = np.array([0.5, 0.25, 2.0], np.float32)
    assert np.allclose(orc.rule_reward(s, w), [1.5, 2.25])
