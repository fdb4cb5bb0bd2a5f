"""One GRPO batch sharded over several GPUs (one process per GPU, torch.distributed).

Rows are independent given the batch's token count N and the advantages, and an advantage needs only
the rewards of its own GRPO group.  So a batch is cut between groups: every rank holds whole groups
(its own packed tokens, cu_seqlens and rewards), and the path needs three exchanges, all of them
all-reduce sums over NCCL:

  1. the int64 count of loss-carrying tokens, before the loss kernel (its coefficients divide by the
     global count); for the sequence-mean aggregation the count of loss-carrying RESPONSES instead
     (rlf_count_live_responses on this rank's responses), the only thing that aggregation needs
     from the other ranks;
  2. the four fp64 loss scalars, after it (each rank's are already divided by the global count, so
     they add up);
  3. for the fused LM-head path, grad_W [V, D] fp32 (the ordinary data-parallel weight-gradient
     all-reduce; grad_hidden and grad_logits stay with the rank that owns the rows).

This module holds the host-side plan (which groups go to which rank) and the three-phase step.  The
kernels are the C-ABI library's, passed in as `ops` (the binding module by default), so the same
step can be driven by any implementation of those calls.
"""
import numpy as np
import torch
import torch.distributed as dist


def plan_shards(cu_seqlens, group_size, world_size):
    """Assign whole GRPO groups to ranks, balancing tokens: groups sorted by token count, largest
    first, each to the least-loaded rank so far (ties: lowest rank), then kept in batch order.

    cu_seqlens: [B+1] response boundaries of the packed batch; response i belongs to group i // group_size.
    -> list over ranks of int64 arrays of response indices (ascending).
    """
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    B = len(cu) - 1
    if group_size <= 0 or world_size <= 0:
        raise ValueError("group_size and world_size must be positive")
    if B % group_size != 0:
        raise ValueError("the batch must hold whole groups (%d responses, groups of %d)" % (B, group_size))
    n_groups = B // group_size
    tokens = np.array([cu[(g + 1) * group_size] - cu[g * group_size] for g in range(n_groups)], dtype=np.int64)
    order = sorted(range(n_groups), key=lambda g: (-int(tokens[g]), g))
    load = [0] * world_size
    mine = [[] for _ in range(world_size)]
    for g in order:
        r = min(range(world_size), key=lambda k: (load[k], k))
        mine[r].append(g)
        load[r] += int(tokens[g])
    out = []
    for r in range(world_size):
        resp = [g * group_size + j for g in sorted(mine[r]) for j in range(group_size)]
        out.append(np.array(resp, dtype=np.int64))
    return out


def take_shard(responses, cu_seqlens, per_token, per_response):
    """Cut one rank's part out of a packed batch (host arrays).
    per_token / per_response: dicts of arrays with leading dimension T resp. B.
    -> (cu_seqlens of the shard, per_token dict, per_response dict)."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    rows = np.concatenate([np.arange(cu[i], cu[i + 1]) for i in responses]) if len(responses) else np.zeros(0, np.int64)
    lens = np.array([cu[i + 1] - cu[i] for i in responses], dtype=np.int64)
    new_cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    return new_cu, {k: v[rows] for k, v in per_token.items()}, {k: v[responses] for k, v in per_response.items()}


def _all_reduce_sum(t, group):
    # issued whenever a group is given, a group of one included: the call is the same for any size
    if group is not None and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


def _ops(ops):
    if ops is None:
        from . import binding as ops          # the CUDA library; raises if it has not been built
    return ops


def count_phase(ids, cu_seqlens, open_id, close_id, ops=None):
    """Phase 1 on this rank's tokens: loss mask, token -> response map and the local count of
    loss-carrying tokens (int64[1], still to be summed over the ranks)."""
    return _ops(ops).rlf_build_loss_mask(ids, cu_seqlens, open_id, close_id)


def loss_phase(n_global, mask, seq_id, ids, rewards, group_size, old_logp, ref_logp, eps_clip, beta_kl, logits=None,
               hidden=None, W=None, grad_W=None, accumulate_grad_W=False, adv_eps=1e-6, ops=None, aggregation=0,
               eps_clip_high=None):
    """Phase 2 on this rank's tokens, against the batch's global count (tokens for the token mean,
    loss-carrying responses for the sequence mean): advantages of this rank's groups, log-probs, this
    rank's share of the loss scalars (they add up over ranks) and gradients (grad_W is this rank's
    contribution, still to be summed over the ranks).  aggregation 1 or an upper clip width of its own
    go through the *_obj entry points."""
    ops = _ops(ops)
    if (logits is None) == (hidden is None):
        raise ValueError("give either logits or hidden + W")
    adv = ops.rlf_group_advantage(rewards, group_size=group_size, eps=adv_eps)
    out = dict(adv=adv)
    if aggregation != 0 or eps_clip_high is not None:
        hi = eps_clip if eps_clip_high is None else eps_clip_high
        if logits is not None:
            logp, loss, grad = ops.rlf_grpo_logp_loss_fwd_bwd_obj(logits, ids, seq_id, adv, old_logp, ref_logp, mask,
                                                                  eps_clip, hi, beta_kl, aggregation=aggregation,
                                                                  denom=n_global)
            out.update(logp=logp, loss=loss, grad_logits=grad)
        else:
            logp, loss, gh, gw = ops.rlf_fused_lmhead_grpo_obj(hidden, W, ids, seq_id, adv, old_logp, ref_logp, mask,
                                                               eps_clip, hi, beta_kl, aggregation=aggregation,
                                                               denom=n_global, grad_W=grad_W,
                                                               accumulate_grad_W=accumulate_grad_W)
            out.update(logp=logp, loss=loss, grad_hidden=gh, grad_W=gw)
        return out
    if logits is not None:
        logp, loss, grad = ops.rlf_grpo_logp_loss_fwd_bwd(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip,
                                                          beta_kl, denom=n_global)
        out.update(logp=logp, loss=loss, grad_logits=grad)
    else:
        logp, loss, gh, gw = ops.rlf_fused_lmhead_grpo(hidden, W, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip,
                                                       beta_kl, denom=n_global, grad_W=grad_W,
                                                       accumulate_grad_W=accumulate_grad_W)
        out.update(logp=logp, loss=loss, grad_hidden=gh, grad_W=gw)
    return out


def sharded_grpo_step(ids, cu_seqlens, rewards, group_size, old_logp, ref_logp, open_id, close_id, eps_clip, beta_kl,
                      logits=None, hidden=None, W=None, grad_W=None, accumulate_grad_W=False, adv_eps=1e-6,
                      group=None, ops=None, reduce_grad_W=True, n_global=None, aggregation=0, eps_clip_high=None):
    """This rank's part of one sharded step.  All tensors are this rank's own (whole groups).

    Give `logits` [T_local, V] for the logits path (returns grad_logits) or `hidden` [T_local, D] and
    `W` [V, D] for the fused LM-head path (returns grad_hidden and the all-reduced grad_W).
    `group`: the process group of the ranks that share the batch (None: no exchange, a single-rank step).
    When grad_W is accumulated over several micro-batches, pass reduce_grad_W=False on all but the
    last one (a reduced buffer must not be reduced again), and pass the whole batch's token count as
    `n_global` (int64[1], e.g. the n_global a counting pass over the whole shard returned): a
    micro-batch's own count is not the batch's denominator.  With `n_global` given the count exchange
    is skipped.  aggregation: 0 = masked token mean over the batch (the exchanged count is of tokens),
    1 = mean over loss-carrying responses of each response's token mean (the exchanged count is of such
    responses); eps_clip_high: upper clip width when it differs from eps_clip.
    -> dict(mask, seq_id, n_local, n_global, adv, logp, loss (global, fp64[4]), grad_logits | grad_hidden, grad_W)
    """
    mask, seq_id, n_local = count_phase(ids, cu_seqlens, open_id, close_id, ops)
    if aggregation == 1:
        n_local = _ops(ops).rlf_count_live_responses(mask, cu_seqlens)
    if n_global is None:
        n_global = _all_reduce_sum(n_local.clone(), group)
    out = loss_phase(n_global, mask, seq_id, ids, rewards, group_size, old_logp, ref_logp, eps_clip, beta_kl,
                     logits=logits, hidden=hidden, W=W, grad_W=grad_W, accumulate_grad_W=accumulate_grad_W,
                     adv_eps=adv_eps, ops=ops, aggregation=aggregation, eps_clip_high=eps_clip_high)
    if "grad_W" in out and reduce_grad_W:
        _all_reduce_sum(out["grad_W"], group)
    out["loss"] = _all_reduce_sum(out["loss"].clone(), group)
    out.update(mask=mask, seq_id=seq_id, n_local=n_local, n_global=n_global)
    return out
