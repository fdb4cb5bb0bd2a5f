"""GPU parity of the forward-only fused LM-head pass (log-prob and entropy from hidden states, logits
never stored) against the fp64 oracle: |d logp| <= 2e-3 as everywhere, entropy to 1e-3 absolute (it is
lse - E[z], both fp32 sums over the vocabulary of bf16-product logits)."""
import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
import gpu_common as gc

pytestmark = pytest.mark.gpu
DEV = "cuda"
ENT_ATOL = 1e-3
SMALL = dict(len_lo=20, len_hi=28, spans_lo=1, spans_hi=2, obs_lo=2, obs_hi=4)


@pytest.fixture(params=[1, 0], ids=["pair", "single"])
def form(request):
    b = gc.binding()
    b.tune_lmhead(request.param)
    yield request.param
    b.tune_lmhead(1)


@pytest.mark.parametrize("V,D,w_std", [(2048, 128, 0.3), (1032, 64, 1.0), (4096 + 264, 192, 0.3), (20488, 256, 0.1)])
def test_fused_logp_entropy_matches_oracle(V, D, w_std, form):
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], V=V, D=D, w_std=w_std, **SMALL)
    batch = synth.make_batch(spec, DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    logp, ent = b.rlf_fused_lmhead_logp_entropy(batch.hidden, batch.W, batch.ids, dev_status=st)
    logp_only, none = b.rlf_fused_lmhead_logp_entropy(batch.hidden, batch.W, batch.ids, want_entropy=False)
    torch.cuda.synchronize()
    assert st.item() == 0 and none is None
    want_lp, want_ent = orc.fused_lmhead_logp_entropy(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W),
                                                      batch.ids.cpu().numpy())
    assert np.abs(logp.cpu().numpy() - want_lp).max() <= gc.LOGP_ATOL
    assert np.abs(ent.cpu().numpy() - want_ent).max() <= ENT_ATOL
    assert torch.equal(logp, logp_only)            # the entropy accumulation does not touch the log-prob
    assert (ent >= 0).all() and (ent <= np.log(V) + 1e-4).all()


def test_fused_logp_entropy_full_vocabulary_reduced_T_and_training_path_agreement():
    """Qwen3-4B head (V = 151936, D = 2560) at 16 x 8 tokens, every column tile and split of the
    full-size sweep; the training entry point's forward returns the same log-probs."""
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], len_lo=8, len_hi=8, spans_lo=1, spans_hi=1, obs_lo=1, obs_hi=2)
    batch = synth.make_batch(spec, DEV)
    logp, ent = b.rlf_fused_lmhead_logp_entropy(batch.hidden, batch.W, batch.ids)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=spec.group_size)
    lp_train, _, _, _ = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp,
                                                mask, synth.EPS_CLIP, synth.BETA_KL, denom=n, want_grad_hidden=False,
                                                want_grad_W=False)
    torch.cuda.synchronize()
    want_lp, want_ent = orc.fused_lmhead_logp_entropy(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W),
                                                      batch.ids.cpu().numpy())
    assert np.abs(logp.cpu().numpy() - want_lp).max() <= gc.LOGP_ATOL
    assert np.abs(ent.cpu().numpy() - want_ent).max() <= ENT_ATOL
    assert (logp - lp_train).abs().max().item() <= 2e-6


def test_fused_logp_entropy_edge_cases():
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], V=2048, D=128, w_std=0.3, **SMALL)
    batch = synth.make_batch(spec, DEV)
    # a zero head: the uniform distribution whatever the hidden states
    W0 = torch.zeros_like(batch.W)
    logp, ent = b.rlf_fused_lmhead_logp_entropy(batch.hidden, W0, batch.ids)
    torch.cuda.synchronize()
    assert (logp + np.log(2048)).abs().max().item() <= 1e-5 and (ent - np.log(2048)).abs().max().item() <= 1e-5
    # ids outside the vocabulary: NaN log-prob, a status bit, the other rows and all entropies unaffected
    ids = batch.ids.clone()
    ids[5], ids[17] = 2048, -3
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    lp2, ent2 = b.rlf_fused_lmhead_logp_entropy(batch.hidden, batch.W, ids, dev_status=st)
    lp1, ent1 = b.rlf_fused_lmhead_logp_entropy(batch.hidden, batch.W, batch.ids)
    torch.cuda.synchronize()
    assert st.item() == b.DEV_BAD_TARGET
    bad = torch.zeros_like(ids, dtype=torch.bool)
    bad[5] = bad[17] = True
    assert torch.isnan(lp2[bad]).all() and torch.equal(lp2[~bad], lp1[~bad]) and torch.equal(ent2, ent1)
    # T = 0
    e = torch.empty((0, 128), dtype=torch.bfloat16, device=DEV)
    lp0, en0 = b.rlf_fused_lmhead_logp_entropy(e, batch.W, torch.empty(0, dtype=torch.int32, device=DEV))
    assert lp0.numel() == 0 and en0.numel() == 0


def test_fused_logp_entropy_peaked_rows():
    """A head row aligned with the hidden state gives that column a dominant logit: entropy near 0,
    log-prob of that column near 0 (the running-maximum rescaling of the entropy sum is exercised)."""
    b = gc.binding()
    T, D, V = 300, 128, 4096 + 264
    g = torch.Generator(device=DEV)
    g.manual_seed(5)
    H = torch.randn((T, D), device=DEV, generator=g).to(torch.bfloat16)
    W = (torch.randn((V, D), device=DEV, generator=g) * 0.05).to(torch.bfloat16)
    ids = torch.randint(0, V, (T,), device=DEV, generator=g).to(torch.int32)
    W[ids.long()] = (H.float() * 0.5).to(torch.bfloat16)       # z_y ~ 0.5 |h|^2 ~ 64; last writer wins on duplicates
    logp, ent = b.rlf_fused_lmhead_logp_entropy(H, W, ids)
    torch.cuda.synchronize()
    want_lp, want_ent = orc.fused_lmhead_logp_entropy(synth.bf16_bits(H), synth.bf16_bits(W), ids.cpu().numpy())
    assert np.abs(logp.cpu().numpy() - want_lp).max() <= gc.LOGP_ATOL
    assert np.abs(ent.cpu().numpy() - want_ent).max() <= ENT_ATOL
    assert want_ent.min() < 1e-6
