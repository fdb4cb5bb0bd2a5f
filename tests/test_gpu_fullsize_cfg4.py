"""Full-size parity of the Qwen3-8B-shaped long-context recipe (T = 65536 = 8 x 8192, D = 4096,
V = 151936), processed the way the recipe words it: 8 micro-batches of one 8192-token response with the
batch's token count as denominator.  Fused LM-head path: grad_W accumulated over the micro-batches;
grad_hidden rows of sampled tokens against the oracle, every row's log-prob and the summed scalar loss
against the oracle run on fp64 logits of the whole batch, grad_W through its zero column sums and against the single-call result.  Logits
path: one micro-batch of bf16 logits formed from the hidden states (the recipe's stand-in for the model's
own head), sampled rows against the oracle."""
import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
import gpu_common as gc
from util import loss_close, ulp_error_bf16
from test_gpu_fused import _close_tensor

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_cfg4_full_size_micro_batched():
    b = gc.binding()
    spec = synth.SPECS[4]
    batch = synth.make_batch(spec, DEV)
    T, MB = batch.T, 8192
    assert (T, spec.D, spec.V) == (65536, 4096, 151936) and batch.rewards.shape[0] == 8
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id, dev_status=st)
    adv = b.rlf_group_advantage(batch.rewards, group_size=spec.group_size, dev_status=st)
    ora = gc.oracle_chain(batch)
    assert np.array_equal(mask.cpu().numpy(), ora["mask"]) and n.item() == ora["n"]
    assert np.abs(adv.cpu().numpy() - ora["adv64"]).max() <= 1e-6

    # fused path, 8 micro-batches
    ws = b.new_workspace(b.FN_FUSED_LMHEAD, MB, spec.V, spec.D, b.RLF_BF16, DEV)
    gh = torch.empty((T, spec.D), dtype=torch.bfloat16, device=DEV)
    gw = torch.empty((spec.V, spec.D), dtype=torch.float32, device=DEV)
    logp = torch.empty(T, dtype=torch.float32, device=DEV)
    loss_sum = torch.zeros(4, dtype=torch.float64, device=DEV)
    loss = torch.empty(4, dtype=torch.float64, device=DEV)
    for i in range(T // MB):
        sl = slice(i * MB, (i + 1) * MB)
        b.rlf_fused_lmhead_grpo(batch.hidden[sl], batch.W, batch.ids[sl], seq[sl], adv, batch.old_logp[sl],
                                batch.ref_logp[sl], mask[sl], synth.EPS_CLIP, synth.BETA_KL, denom=n, grad_hidden=gh[sl],
                                grad_W=gw, accumulate_grad_W=i > 0, logp_out=logp[sl], loss_out=loss, workspace=ws,
                                dev_status=st)
        loss_sum += loss
    torch.cuda.synchronize()
    assert st.item() == 0

    rng = np.random.default_rng(4)
    live = np.flatnonzero(ora["mask"])
    rows = np.unique(np.concatenate([[0, MB - 1, MB, T - 1], rng.choice(live, size=16, replace=False),
                                     rng.integers(0, T, size=4)]))
    rt = torch.as_tensor(rows, device=DEV)
    r = orc.fused_lmhead_grpo(synth.bf16_bits(batch.hidden[rt]), synth.bf16_bits(batch.W), batch.ids.cpu().numpy()[rows],
                              ora["seq_id"][rows], ora["adv"], batch.old_logp.cpu().numpy()[rows],
                              batch.ref_logp.cpu().numpy()[rows], ora["mask"][rows], synth.EPS_CLIP, synth.BETA_KL,
                              denom=ora["n"], want_grad_hidden=True, want_grad_W=False)
    assert np.abs(logp[rt].cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
    _close_tensor(gh[rt].float().cpu().numpy(), r["grad_hidden"], "grad_hidden rows")
    assert not gh[~mask.bool()].any()

    # every row of all eight micro-batches: log-prob and the summed scalar loss against the oracle
    # (fp64 logits from the library's fp64 contraction, then the oracle's loss)
    logp_o, loss_o, coef_o = gc.oracle_all_rows_through_fp64_head(batch.hidden, batch.W, ora, batch.old_logp.cpu().numpy(),
                                                                  batch.ref_logp.cpu().numpy(), row_chunk=2048,
                                                                  want_coef=True)
    assert np.abs(logp.cpu().numpy() - logp_o).max() <= gc.LOGP_ATOL
    # rows of the accumulated grad_W (a sum over all eight micro-batches) against the oracle's per-row outputs
    vs = np.unique(np.concatenate([ora["ids"][live][:12], rng.integers(0, spec.V, size=12), [spec.V - 1]]))
    gw_o = gc.oracle_grad_W_rows(batch.hidden, batch.W, batch.ids, logp_o, coef_o, vs)
    _close_tensor(gw[torch.as_tensor(vs, device=DEV)].cpu().numpy(), gw_o, "grad_W rows")
    assert np.abs(logp_o[rows] - r["logp"]).max() <= 1e-9
    floor = gc.loss_floor(ora)
    ls = loss_sum.cpu().numpy()
    for k in range(3):
        assert loss_close(ls[k], loss_o[k], floor if k < 2 else 1e-9, gc.LOSS_RTOL), (k, ls, loss_o)

    col = gw.double().sum(dim=0).abs().max().item()
    assert col <= 1e-3 * gw.double().abs().sum(dim=0).max().item()

    # the same batch in one call: same log-probs to rounding, same weight gradient to the per-tensor tolerance
    ws1 = b.new_workspace(b.FN_FUSED_LMHEAD, T, spec.V, spec.D, b.RLF_BF16, DEV)
    gw1 = torch.empty_like(gw)
    logp1, loss1, gh1, _ = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp,
                                                   batch.ref_logp, mask, synth.EPS_CLIP, synth.BETA_KL, denom=n,
                                                   grad_W=gw1, workspace=ws1, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert (logp1 - logp).abs().max().item() <= 1e-4
    assert loss_close(loss1[0].item(), loss_sum[0].item(), floor, gc.LOSS_RTOL)
    assert (gw1 - gw).abs().max().item() <= 2.0 ** -7 * gw1.abs().max().item()
    assert (gh1.float() - gh.float()).abs().max().item() <= 2.0 ** -7 * gh1.float().abs().max().item()
    del ws, ws1, gw, gw1, gh, gh1
    torch.cuda.empty_cache()

    # logits path on the last micro-batch: bf16 logits formed from the hidden states
    sl = slice(T - MB, T)
    logits = torch.matmul(batch.hidden[sl], batch.W.t())
    lp2, loss2, grad = b.rlf_grpo_logp_loss_fwd_bwd(logits, batch.ids[sl], seq[sl], adv, batch.old_logp[sl],
                                                    batch.ref_logp[sl], mask[sl], synth.EPS_CLIP, synth.BETA_KL, denom=n,
                                                    dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    rows2 = np.sort(rng.choice(MB, size=400, replace=False))
    g_rows = (T - MB) + rows2
    r2 = orc.grpo_loss(gc.to_np(logits[torch.as_tensor(rows2, device=DEV)]), batch.ids.cpu().numpy()[g_rows],
                       ora["seq_id"][g_rows], ora["adv"], batch.old_logp.cpu().numpy()[g_rows],
                       batch.ref_logp.cpu().numpy()[g_rows], ora["mask"][g_rows], synth.EPS_CLIP, synth.BETA_KL,
                       denom=ora["n"])
    assert np.abs(lp2.cpu().numpy()[rows2] - r2["logp"]).max() <= gc.LOGP_ATOL
    guard = gc.near_clip_bound(r2["logp"], batch.old_logp.cpu().numpy()[g_rows], None)
    got = gc.grad_to_f64(grad[torch.as_tensor(rows2, device=DEV)])
    assert ulp_error_bf16(got[~guard], r2["grad"][~guard]).max() <= gc.GRAD_ULPS
    assert not grad[~mask[sl].bool()].any()
