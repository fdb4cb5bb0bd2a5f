"""GPU parity of the KL-in-reward variant (rlf_kl_in_reward) against the oracle: the summed
estimate and the adjusted reward of every response to one fp32 rounding, on the ragged recipe and on
edge cases (empty responses, all-masked responses, a malformed cu_seqlens)."""
import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
import gpu_common as gc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _tokens(cfg, **kw):
    spec = synth.scaled(synth.SPECS[cfg], **kw)
    tok = synth.make_tokens(spec)
    rng = np.random.default_rng(77 + cfg)
    T = len(tok.ids)
    old = rng.normal(-2.0, 1.0, size=T).astype(np.float32)
    ref = (old + rng.normal(0.0, 0.1, size=T)).astype(np.float32)
    return spec, tok, old, ref


@pytest.mark.parametrize("cfg,kw", [(2, {}), (4, {}), (0, {}),
                                    (1, dict(num_prompts=1, group_size=3, len_lo=9, len_hi=9, spans_lo=1, spans_hi=1, obs_lo=1, obs_hi=2))])
@pytest.mark.parametrize("kind", [0, 1, 2])
def test_kl_in_reward_matches_oracle(cfg, kw, kind):
    b = gc.binding()
    spec, tok, old, ref = _tokens(cfg, **kw)
    ids = torch.from_numpy(tok.ids).to(DEV)
    cu = torch.from_numpy(tok.cu_seqlens).to(DEV)
    mask, _, _ = b.rlf_build_loss_mask(ids, cu, spec.open_id, spec.close_id)
    rewards = torch.from_numpy(tok.rewards).to(DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    beta = 0.05
    got, kl = b.rlf_kl_in_reward(rewards, torch.from_numpy(old).to(DEV), torch.from_numpy(ref).to(DEV), mask, cu,
                                 beta, kind, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    want, want_kl = orc.kl_in_reward(tok.rewards, old, ref, mask.cpu().numpy(), tok.cu_seqlens, beta, kind)
    # fp64 sums rounded once to fp32 (the CPU and the GPU add in different orders: a few fp64 ulps)
    assert np.abs(kl.cpu().numpy() - want_kl).max() <= 1e-7 * max(np.abs(want_kl).max(), 1e-30) + 1e-12
    assert np.abs(got.cpu().numpy() - want).max() <= 1e-7 * np.abs(want).max() + 1e-12
    # the adjusted rewards feed the advantage
    adv = b.rlf_group_advantage(got, group_size=spec.group_size)
    torch.cuda.synchronize()
    want_adv = orc.group_advantage(got.cpu().numpy(), group_size=spec.group_size)
    assert np.allclose(adv.cpu().numpy(), want_adv, rtol=2e-6, atol=1e-30)


def test_kl_in_reward_edge_cases():
    b = gc.binding()
    # responses: empty, all masked, one token; then a malformed boundary
    cu = np.array([0, 0, 4, 5], np.int32)
    mask = np.array([0, 0, 0, 0, 1], np.uint8)
    old = np.array([-1.0, -2.0, -3.0, -4.0, -1.5], np.float32)
    ref = np.array([-1.5, -2.5, -2.0, -4.0, -1.0], np.float32)
    r = np.array([0.25, 0.5, 1.0], np.float32)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    for kind in (0, 1, 2):
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        got, kl = b.rlf_kl_in_reward(dev(r), dev(old), dev(ref), dev(mask), dev(cu), 0.5, kind, dev_status=st)
        torch.cuda.synchronize()
        want, want_kl = orc.kl_in_reward(r, old, ref, mask, cu, 0.5, kind)
        assert st.item() == 0
        assert np.array_equal(got.cpu().numpy()[:2], r[:2]) and np.all(kl.cpu().numpy()[:2] == 0)
        assert np.allclose(got.cpu().numpy(), want, rtol=1e-7) and np.allclose(kl.cpu().numpy(), want_kl, rtol=1e-7)
    # in place over the rewards
    rr = dev(r)
    b.rlf_kl_in_reward(rr, dev(old), dev(ref), dev(mask), dev(cu), 0.5, 2, reward_out=rr)
    torch.cuda.synchronize()
    assert np.allclose(rr.cpu().numpy(), orc.kl_in_reward(r, old, ref, mask, cu, 0.5, 2)[0], rtol=1e-7)
    # a boundary beyond T is reported and clipped, nothing out of bounds is read
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    bad = np.array([0, 2, 9, 5], np.int32)
    got, _ = b.rlf_kl_in_reward(dev(r), dev(old), dev(ref), dev(mask), dev(bad), 0.5, 0, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() & b.DEV_BAD_SEQ
    assert np.isfinite(got.cpu().numpy()).all()
    with pytest.raises(Exception):
        b.rlf_kl_in_reward(dev(r), dev(old), dev(ref), dev(mask), dev(cu), 0.5, 7)
