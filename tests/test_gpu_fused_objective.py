"""GPU parity of the fused LM-head call under the objective variants (asymmetric clip range,
sequence-mean aggregation) and of its skip-masked form, against the fp64 oracle, with the tolerances of
the base fused entry point."""
import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
import gpu_common as gc
from util import loss_close
from test_gpu_fused import _close_tensor

pytestmark = pytest.mark.gpu
DEV = "cuda"
SMALL = dict(len_lo=20, len_hi=28, spans_lo=1, spans_hi=2, obs_lo=2, obs_hi=4)


def _setup(V, D):
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], V=V, D=D, w_std=0.3, **SMALL)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    return b, spec, batch, mask, seq, n, adv


@pytest.mark.parametrize("V,D,lo,hi,agg,skip", [(2048, 128, 0.2, 0.28, 0, 0), (2048, 128, 0.2, 0.28, 1, 0),
                                                 (1032, 64, 0.05, 0.1, 1, 1), (4096 + 264, 192, 0.1, 0.4, 0, 1)])
def test_fused_objective_variants_match_oracle(V, D, lo, hi, agg, skip):
    b, spec, batch, mask, seq, n, adv = _setup(V, D)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    beta = 0.02
    logp, loss, gh, gw = b.rlf_fused_lmhead_grpo_obj(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp,
                                                     batch.ref_logp, mask, lo, hi, beta, aggregation=agg,
                                                     skip_masked=bool(skip), denom=n if agg == 0 else None,
                                                     dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    m = mask.cpu().numpy()
    r = orc.fused_lmhead_grpo_obj(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W), batch.ids.cpu().numpy(),
                                  seq.cpu().numpy(), adv.cpu().numpy(), batch.old_logp.cpu().numpy(),
                                  batch.ref_logp.cpu().numpy(), m, lo, hi, beta, aggregation=agg)
    lp = logp.cpu().numpy()
    if skip:
        assert np.isnan(lp[m == 0]).all()
        assert np.abs(lp[m == 1] - r["logp"][m == 1]).max() <= gc.LOGP_ATOL
    else:
        assert np.abs(lp - r["logp"]).max() <= gc.LOGP_ATOL
    lg = loss.cpu().numpy()
    # The surrogate's mean nearly cancels here (zero-mean advantages, ratios near 1), so a tolerance
    # relative to its value alone would ask for more than fp32 log-probs can give: a log-prob error e
    # moves a token's term by |A| rho e.  Floor of the scale: the mean |A| of the unmasked tokens times the
    # log-prob tolerance.
    a_tok = np.abs(adv.cpu().numpy()[seq.cpu().numpy()])[m == 1]
    floor = gc.LOGP_ATOL * float(a_tok.mean()) if a_tok.size else 1e-6
    for k in range(3):
        assert loss_close(lg[k], r["loss"][k], floor if k < 2 else 1e-6, gc.LOSS_RTOL), (k, lg, r["loss"])
    assert abs(lg[3] - r["loss"][3]) <= 2.0 / max(int(m.sum()), 1)
    _close_tensor(gh.float().cpu().numpy(), r["grad_hidden"], "grad_hidden")
    _close_tensor(gw.cpu().numpy(), r["grad_W"], "grad_W")
    assert not gh[mask == 0].any()


def test_fused_symmetric_token_mean_variant_is_the_base_entry_point():
    b, spec, batch, mask, seq, n, adv = _setup(2048, 128)
    args = (batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask)
    lp0, l0, gh0, gw0 = b.rlf_fused_lmhead_grpo(*args, synth.EPS_CLIP, synth.BETA_KL, denom=n)
    lp1, l1, gh1, gw1 = b.rlf_fused_lmhead_grpo_obj(*args, synth.EPS_CLIP, synth.EPS_CLIP, synth.BETA_KL, denom=n)
    torch.cuda.synchronize()
    assert torch.equal(lp0, lp1) and torch.equal(l0, l1) and torch.equal(gh0, gh1) and torch.equal(gw0, gw1)


@pytest.mark.parametrize("bwd", [True, False])
def test_fused_skip_masked_changes_only_the_masked_log_probs(bwd):
    """Loss, gradients and the unmasked rows' log-probs are bit-identical with and without skipping."""
    b, spec, batch, mask, seq, n, adv = _setup(4096 + 264, 192)
    args = (batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask, 0.2, 0.2, synth.BETA_KL)
    kw = dict(denom=n, want_grad_hidden=bwd, want_grad_W=bwd)
    lp0, l0, gh0, gw0 = b.rlf_fused_lmhead_grpo_obj(*args, skip_masked=False, **kw)
    lp1, l1, gh1, gw1 = b.rlf_fused_lmhead_grpo_obj(*args, skip_masked=True, **kw)
    torch.cuda.synchronize()
    live = mask == 1
    assert torch.isnan(lp1[~live]).all() and not torch.isnan(lp0).any()
    if bwd:
        assert torch.equal(lp0[live], lp1[live])
        assert torch.equal(gh0, gh1) and torch.equal(gw0, gw1)
        assert torch.equal(l0, l1)
    else:
        # forward only without skipping sweeps all rows in one launch (different split boundaries per row tile
        # are the same, but the rows sit in other tiles): equal to fp32 rounding, not bitwise
        assert (lp0[live] - lp1[live]).abs().max().item() <= 1e-5
        assert abs(l0[0].item() - l1[0].item()) <= 1e-6 * max(abs(l0[0].item()), 1e-6)


def test_fused_objective_all_rows_masked_and_bad_arguments():
    b, spec, batch, mask, seq, n, adv = _setup(1032, 64)
    zero = torch.zeros_like(mask)
    logp, loss, gh, gw = b.rlf_fused_lmhead_grpo_obj(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp,
                                                     batch.ref_logp, zero, 0.2, 0.3, 0.01, aggregation=1,
                                                     skip_masked=True)
    torch.cuda.synchronize()
    assert torch.isnan(logp).all() and loss[0].item() == 0.0 and not gh.any() and not gw.any()
    with pytest.raises(Exception):
        b.rlf_fused_lmhead_grpo_obj(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                    0.2, 0.3, 0.01, aggregation=2)


def test_fused_results_do_not_depend_on_the_schedule():
    """Scheduling block, worker cap and backward chunk are tuning choices: log-probs, loss and
    grad_hidden are bit-identical for every setting; grad_W is bit-identical unless the chunking
    changes (then the chunks' contributions are added in another order: fp32 rounding only)."""
    b, spec, batch, mask, seq, n, adv = _setup(4096 + 264, 192)
    # enough rows for several token tiles and, with 2-tile chunks, several chunks
    spec = synth.scaled(spec, len_lo=60, len_hi=60)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    args = (batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask, synth.EPS_CLIP, synth.BETA_KL)
    outs = {}
    try:
        for key in ((0, 0, 0), (1, 0, 0), (3, 5, 0), (1000, 1, 0), (0, 0, 2), (2, 7, 4)):
            b.tune_lmhead_schedule(*key)
            outs[key] = b.rlf_fused_lmhead_grpo(*args, denom=n)
            torch.cuda.synchronize()
    finally:
        b.tune_lmhead_schedule(0, 0, 0)
    # pacing (the workers' meeting points before each unit) only delays loads
    try:
        b.tune_lmhead_pacing(0)
        unpaced = b.rlf_fused_lmhead_grpo(*args, denom=n)
        torch.cuda.synchronize()
    finally:
        b.tune_lmhead_pacing(1)
    for got, want in zip(unpaced, outs[(0, 0, 0)]):
        assert torch.equal(got, want)
    ref = outs[(0, 0, 0)]
    for key, o in outs.items():
        assert torch.equal(o[0], ref[0]) and torch.equal(o[1], ref[1]) and torch.equal(o[2], ref[2]), key
        if key[2] == 0:
            assert torch.equal(o[3], ref[3]), key
        else:
            assert (o[3] - ref[3]).abs().max().item() <= 1e-5 * ref[3].abs().max().item(), key


@pytest.mark.parametrize("tokens", [24, 44, 60])
def test_two_accumulator_gradient_contractions_are_bit_identical_to_the_one_accumulator_form(tokens):
    """In pair form the two gradient contractions give each CTA pair two 256-row tiles per 256-column
    slab.  Every output element is still one fp32 accumulation over the same k-slabs in the same order,
    so both forms must agree bit for bit: at tile counts that leave the last unit with one, two or three
    of its four tiles, with several chunks, and when grad_W is accumulated onto given values (a vector
    reduction in one form's drain against a plain store in the first chunk)."""
    b, spec, batch, mask, seq, n, adv = _setup(4096 + 264, 192)
    spec = synth.scaled(spec, len_lo=tokens, len_hi=tokens)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    args = (batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask, synth.EPS_CLIP, synth.BETA_KL)
    gw0 = torch.randn((spec.V, spec.D), device=DEV)
    outs = {}
    try:
        for acc2 in (1, 0):
            for chunk in (0, 2, 6):
                for accumulate in (False, True):
                    b.tune_lmhead_backward(1, acc2)
                    b.tune_lmhead_schedule(0, 0, chunk)
                    outs[(acc2, chunk, accumulate)] = b.rlf_fused_lmhead_grpo(
                        *args, denom=n, grad_W=gw0.clone() if accumulate else None, accumulate_grad_W=accumulate)
                    torch.cuda.synchronize()
    finally:
        b.tune_lmhead_backward(1, 1)
        b.tune_lmhead_schedule(0, 0, 0)
    for (acc2, chunk, accumulate), o in outs.items():
        ref = outs[(0, chunk, accumulate)]
        for got, want in zip(o, ref):
            assert torch.equal(got, want), (acc2, chunk, accumulate)


def test_fused_repeated_calls_reproduce_the_first_bit_for_bit():
    """Twenty calls over the same inputs on the Qwen3-4B head shape (full V and D, 1536 tokens: several
    token tiles, all 74 CTA pairs busy, workers paced by a device counter): log-probs, loss, grad_hidden
    and, within one backward chunk, grad_W come out with the same bits every time."""
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], len_lo=96, len_hi=96, spans_lo=1, spans_hi=2, obs_lo=4, obs_hi=12)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    first = None
    for _ in range(20):
        out = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                      synth.EPS_CLIP, synth.BETA_KL, denom=n, dev_status=st)
        cur = [o.clone() for o in out]
        if first is None:
            first = cur
        else:
            assert all(torch.equal(x, y) for x, y in zip(cur, first))
    assert st.item() == 0
