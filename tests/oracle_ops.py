"""A stand-in for the CUDA binding, backed by the CPU oracle, with the binding's call signatures (torch
tensors in and out).  TEST INFRASTRUCTURE: it lets the multi-rank step logic run as gloo ranks on
hosts without a GPU; the product never imports it."""
import numpy as np
import torch

from oracle import rlf_oracle as orc


def rlf_build_loss_mask(ids, cu_seqlens, open_id, close_id, **_):
    m, s, n = orc.build_loss_mask(ids.numpy(), cu_seqlens.numpy(), open_id, close_id)
    return torch.from_numpy(m), torch.from_numpy(s), torch.tensor([n], dtype=torch.int64)


def rlf_group_advantage(rewards, group_size=None, eps=1e-6, **_):
    return torch.from_numpy(orc.group_advantage(rewards.numpy(), group_size=group_size, eps=eps).astype(np.float32))


def rlf_grpo_logp_loss_fwd_bwd(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip, beta_kl, denom=None, **_):
    r = orc.grpo_loss(logits.double().numpy(), ids.numpy(), seq_id.numpy(), adv.numpy(), old_logp.numpy(),
                      ref_logp.numpy(), mask.numpy(), eps_clip, beta_kl, denom=None if denom is None else int(denom.item()))
    return torch.from_numpy(r["logp"]), torch.from_numpy(r["loss"]), torch.from_numpy(r["grad"])


def rlf_fused_lmhead_grpo(hidden, W, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip, beta_kl, denom=None,
                          grad_W=None, accumulate_grad_W=False, **_):
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    r = orc.fused_lmhead_grpo(bits(hidden), bits(W), ids.numpy(), seq_id.numpy(), adv.numpy(), old_logp.numpy(),
                              ref_logp.numpy(), mask.numpy(), eps_clip, beta_kl,
                              denom=None if denom is None else int(denom.item()))
    gw = torch.from_numpy(r["grad_W"])
    if grad_W is not None:
        if accumulate_grad_W:
            grad_W += gw
        else:
            grad_W.copy_(gw)
        gw = grad_W
    return torch.from_numpy(r["logp"]), torch.from_numpy(r["loss"]), torch.from_numpy(r["grad_hidden"]), gw


def rlf_count_live_responses(mask, cu_seqlens, **_):
    m, cu = mask.numpy(), cu_seqlens.numpy()
    return torch.tensor([sum(1 for b in range(len(cu) - 1) if m[cu[b]:cu[b + 1]].any())], dtype=torch.int64)


def rlf_grpo_logp_loss_fwd_bwd_obj(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_low, eps_high, beta_kl,
                                   aggregation=0, denom=None, **_):
    r = orc.grpo_loss_obj(logits.double().numpy(), ids.numpy(), seq_id.numpy(), adv.numpy(), old_logp.numpy(),
                          ref_logp.numpy(), mask.numpy(), eps_low, eps_high, beta_kl, aggregation=aggregation,
                          denom=None if denom is None else int(denom.item()))
    return torch.from_numpy(r["logp"]), torch.from_numpy(r["loss"]), torch.from_numpy(r["grad"])
