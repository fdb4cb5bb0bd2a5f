"""GPU parity of the objective variants (asymmetric clip range, sequence-mean aggregation) against
the oracle, with the tolerances of the base entry point."""
import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
import gpu_common as gc
from util import loss_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("V,dtype,lo,hi,agg", [(151936, "bf16", 0.2, 0.28, 0), (151936, "bf16", 0.2, 0.28, 1),
                                                 (4096, "bf16", 0.05, 0.1, 1), (1024, "f32", 0.2, 0.3, 1),
                                                 (1001, "bf16", 0.1, 0.1, 1), (200000, "bf16", 0.2, 0.28, 1),
                                                 (262144, "bf16", 0.2, 0.2, 1)])
def test_objective_variants_match_oracle(V, dtype, lo, hi, agg):
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[2], V=V, logits_dtype=dtype, num_prompts=2, group_size=4, len_lo=10, len_hi=60,
                        spans_lo=1, spans_hi=2, cover_lo=0.2, cover_hi=0.5)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=spec.group_size)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    beta = 0.02
    logp, loss, grad = b.rlf_grpo_logp_loss_fwd_bwd_obj(batch.logits, batch.ids, seq, adv, batch.old_logp * 1.0,
                                                        batch.ref_logp, mask, lo, hi, beta, aggregation=agg,
                                                        denom=n if agg == 0 else None, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    r = orc.grpo_loss_obj(gc.to_np(batch.logits), batch.ids.cpu().numpy(), seq.cpu().numpy(), adv.cpu().numpy(),
                          batch.old_logp.cpu().numpy(), batch.ref_logp.cpu().numpy(), mask.cpu().numpy(), lo, hi, beta,
                          aggregation=agg, want_coef=True)
    assert np.abs(logp.cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
    lg = loss.cpu().numpy()
    for k in range(3):
        assert loss_close(lg[k], r["loss"][k], 1e-6, gc.LOSS_RTOL), (k, lg, r["loss"])
    assert abs(lg[3] - r["loss"][3]) <= 2.0 / max(int(mask.sum().item()), 1)
    g = gc.grad_to_f64(grad)
    rho = np.exp(r["logp"] - batch.old_logp.cpu().numpy().astype(np.float64))
    guard = (np.abs(rho - (1 + hi)) < gc.CLIP_GUARD) | (np.abs(rho - (1 - lo)) < gc.CLIP_GUARD)
    ids_np = batch.ids.cpu().numpy()
    if dtype == "f32":
        assert (np.abs(g[~guard] - r["grad"][~guard]) <= 1e-4 * np.abs(r["grad"][~guard]) + 1e-12).all()
    ulps = gc.grad_ulps(g[~guard], r["grad"][~guard], ids_np[~guard], r["coef"][~guard])
    assert ulps.max() <= gc.GRAD_ULPS
    assert (g[mask.cpu().numpy() == 0] == 0).all()


def test_symmetric_token_mean_variant_is_the_base_entry_point():
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[1], len_lo=20, len_hi=20, spans_lo=1, spans_hi=1, obs_lo=2, obs_hi=4)
    batch = synth.make_batch(spec, DEV)
    base = gc.gpu_chain(batch, batch.logits)
    logp, loss, grad = b.rlf_grpo_logp_loss_fwd_bwd_obj(batch.logits, batch.ids, base["seq_id"], base["adv"],
                                                        batch.old_logp, batch.ref_logp, base["mask"], synth.EPS_CLIP,
                                                        synth.EPS_CLIP, synth.BETA_KL, aggregation=0, denom=base["n"])
    torch.cuda.synchronize()
    assert torch.equal(logp, base["logp"]) and torch.equal(loss, base["loss"]) and torch.equal(grad, base["grad"])


def test_sequence_mean_micro_batches_add_up():
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[1], len_lo=24, len_hi=24, spans_lo=1, spans_hi=2, obs_lo=2, obs_hi=5, V=32768)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=spec.group_size)
    full = b.rlf_grpo_logp_loss_fwd_bwd_obj(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                            0.2, 0.28, 0.01, aggregation=1)
    torch.cuda.synchronize()
    S = torch.tensor([batch.B], dtype=torch.int64, device=DEV)
    total = 0.0
    cu = batch.cu_seqlens.cpu().numpy()
    for i in range(0, batch.B, 4):
        a, e = int(cu[i]), int(cu[i + 4])
        part = b.rlf_grpo_logp_loss_fwd_bwd_obj(batch.logits[a:e], batch.ids[a:e], seq[a:e], adv, batch.old_logp[a:e],
                                                batch.ref_logp[a:e], mask[a:e], 0.2, 0.28, 0.01, aggregation=1, denom=S)
        torch.cuda.synchronize()
        total += part[1][0].item()
        assert torch.equal(part[2], full[2][a:e])
    assert abs(total - full[1][0].item()) <= 1e-12 + 1e-9 * abs(total)
