"""The skip-masked variant against the ordinary entry point and the oracle: live rows' log-probs,
gradients and the loss are identical; skipped rows get NaN log-probs and zero (or untouched)
gradient rows."""
import numpy as np
import pytest
import torch

from paper_2509_06980_b200 import synth
import gpu_common as gc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(spec):
    b = gc.binding()
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    return b, batch, mask, seq, n, adv


@pytest.mark.parametrize("V,dtype,L", [(151936, "bf16", 40), (32768, "bf16", 300), (1001, "bf16", 30), (1024, "f32", 30),
                                       (200000, "bf16", 24), (262144, "bf16", 24)])
def test_skip_masked_equals_full_processing_on_live_rows(V, dtype, L):
    spec = synth.scaled(synth.SPECS[1], V=V, logits_dtype=dtype, len_lo=L, len_hi=L, spans_lo=1, spans_hi=3,
                        obs_lo=3, obs_hi=max(4, L // 6))
    b, batch, mask, seq, n, adv = _inputs(spec)
    full = b.rlf_grpo_logp_loss_fwd_bwd(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                        synth.EPS_CLIP, synth.BETA_KL, denom=n)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    grad = torch.full_like(batch.logits, 5.0)
    skip = b.rlf_grpo_logp_loss_fwd_bwd_skip_masked(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp,
                                                    mask, synth.EPS_CLIP, synth.BETA_KL, denom=n, grad_logits=grad,
                                                    dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    m = mask.bool()
    assert 0 < m.sum().item() < batch.T
    assert torch.equal(skip[0][m], full[0][m]) and torch.isnan(skip[0][~m]).all()
    assert torch.equal(skip[1], full[1])
    assert torch.equal(skip[2], full[2])            # live rows identical, skipped rows zero in both
    # against the oracle as well
    ora = gc.oracle_chain(batch, gc.to_np(batch.logits))
    from util import loss_close
    assert loss_close(skip[1][0].item(), ora["loss"][0], 1e-6, gc.LOSS_RTOL)
    lp = skip[0].cpu().numpy()
    assert np.abs(lp[ora["mask"] == 1] - ora["logp"][ora["mask"] == 1]).max() <= gc.LOGP_ATOL


def test_skip_masked_leaves_rows_untouched_when_asked_and_counts_its_own_denominator():
    spec = synth.scaled(synth.SPECS[1], len_lo=24, len_hi=24, spans_lo=1, spans_hi=2, obs_lo=3, obs_hi=5)
    b, batch, mask, seq, n, adv = _inputs(spec)
    full = b.rlf_grpo_logp_loss_fwd_bwd(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                        synth.EPS_CLIP, synth.BETA_KL, denom=n)
    grad = torch.full_like(batch.logits, 5.0)
    skip = b.rlf_grpo_logp_loss_fwd_bwd_skip_masked(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp,
                                                    mask, synth.EPS_CLIP, synth.BETA_KL, denom=None, grad_logits=grad,
                                                    zero_masked_grad=False)
    torch.cuda.synchronize()
    m = mask.bool()
    assert torch.equal(skip[2][m], full[2][m]) and (skip[2][~m] == 5.0).all()
    assert torch.equal(skip[1], full[1])
    # in place, twice in a row on fresh copies: same result (the compaction order may differ)
    for _ in range(2):
        z = batch.logits.clone()
        again = b.rlf_grpo_logp_loss_fwd_bwd_skip_masked(z, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                                         synth.EPS_CLIP, synth.BETA_KL, denom=n, in_place=True)
        torch.cuda.synchronize()
        assert torch.equal(again[2], full[2]) and torch.equal(again[1], full[1])


def test_skip_masked_all_masked_and_none_masked():
    spec = synth.scaled(synth.SPECS[1], len_lo=16, len_hi=16, spans_lo=1, spans_hi=1, obs_lo=2, obs_hi=3, V=16384)
    b, batch, mask, seq, n, adv = _inputs(spec)
    for fill in (0, 1):
        mk = torch.full_like(mask, fill)
        full = b.rlf_grpo_logp_loss_fwd_bwd(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mk,
                                            synth.EPS_CLIP, synth.BETA_KL)
        skip = b.rlf_grpo_logp_loss_fwd_bwd_skip_masked(batch.logits, batch.ids, seq, adv, batch.old_logp,
                                                        batch.ref_logp, mk, synth.EPS_CLIP, synth.BETA_KL)
        torch.cuda.synchronize()
        assert torch.equal(skip[1], full[1]) and torch.equal(skip[2], full[2])
        if fill:
            assert torch.equal(skip[0], full[0])
        else:
            assert torch.isnan(skip[0]).all()
