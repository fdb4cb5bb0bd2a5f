"""The sharded single-batch step with the CUDA kernels on one GPU: the two ranks' shards are run one
after the other (no kernel waits on another), the token counts are summed as the all-reduce would, and
the parts must add up to the unsharded call: loss scalars, row gradients (bit-identical: a row's
gradient depends on the row and the global count only) and the weight gradient."""
import numpy as np
import pytest
import torch

from paper_2509_06980_b200 import sharded, synth
import gpu_common as gc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _shard_inputs(batch, responses, with_head):
    tok = {"ids": batch.ids.cpu().numpy(), "old": batch.old_logp.cpu().numpy(), "ref": batch.ref_logp.cpu().numpy(),
           "rows": np.arange(batch.T)}
    cu, t, r = sharded.take_shard(responses, batch.cu_seqlens.cpu().numpy(), tok, {"rewards": batch.rewards.cpu().numpy()})
    rows = torch.from_numpy(t["rows"]).to(DEV)
    d = dict(ids=torch.from_numpy(t["ids"]).to(DEV), cu=torch.from_numpy(cu).to(DEV),
             rewards=torch.from_numpy(r["rewards"]).to(DEV), old=torch.from_numpy(t["old"]).to(DEV),
             ref=torch.from_numpy(t["ref"]).to(DEV), rows=rows)
    if with_head:
        d["hidden"] = batch.hidden[rows].contiguous()
    else:
        d["logits"] = batch.logits[rows].contiguous()
    return d


@pytest.mark.parametrize("world", [2, 3])
def test_logits_path_shards_add_up(world):
    spec = synth.scaled(synth.SPECS[2], V=4096, num_prompts=4, group_size=4, len_lo=10, len_hi=80, spans_lo=1,
                        spans_hi=2, cover_lo=0.2, cover_hi=0.5)
    batch = synth.make_batch(spec, DEV)
    full = sharded.sharded_grpo_step(batch.ids, batch.cu_seqlens, batch.rewards, spec.group_size, batch.old_logp,
                                     batch.ref_logp, spec.open_id, spec.close_id, synth.EPS_CLIP, synth.BETA_KL,
                                     logits=batch.logits)                      # world of one: no exchange
    ref = gc.gpu_chain(batch, batch.logits)
    assert torch.equal(full["loss"], ref["loss"]) and torch.equal(full["grad_logits"], ref["grad"])
    plan = sharded.plan_shards(batch.cu_seqlens.cpu().numpy(), spec.group_size, world)
    parts = [_shard_inputs(batch, p, False) for p in plan]
    counted = [sharded.count_phase(p["ids"], p["cu"], spec.open_id, spec.close_id) for p in parts]
    n_global = sum(c[2] for c in counted)                                       # what the all-reduce yields
    assert n_global.item() == ref["n"].item()
    loss = torch.zeros(4, dtype=torch.float64, device=DEV)
    for k, (p, (mask, seq, _)) in enumerate(zip(parts, counted)):
        o = sharded.loss_phase(n_global, mask, seq, p["ids"], p["rewards"], spec.group_size, p["old"], p["ref"],
                               synth.EPS_CLIP, synth.BETA_KL, logits=p["logits"])
        torch.cuda.synchronize()
        loss += o["loss"]
        assert torch.equal(o["grad_logits"], ref["grad"][p["rows"]])
        assert torch.equal(o["logp"], ref["logp"][p["rows"]])
        assert torch.equal(o["adv"], ref["adv"][torch.from_numpy(plan[k]).to(DEV)])
    assert torch.allclose(loss, ref["loss"], rtol=1e-12, atol=1e-15)


def test_fused_path_shards_add_up():
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], V=4096 + 264, D=192, w_std=0.3, num_prompts=4, group_size=2, len_lo=24, len_hi=40,
                        spans_lo=1, spans_hi=2, obs_lo=2, obs_hi=4)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=spec.group_size)
    lp, ls, gh, gw = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp,
                                             mask, synth.EPS_CLIP, synth.BETA_KL, denom=n)
    plan = sharded.plan_shards(batch.cu_seqlens.cpu().numpy(), spec.group_size, 2)
    parts = [_shard_inputs(batch, p, True) for p in plan]
    counted = [sharded.count_phase(p["ids"], p["cu"], spec.open_id, spec.close_id) for p in parts]
    n_global = sum(c[2] for c in counted)
    loss = torch.zeros(4, dtype=torch.float64, device=DEV)
    gw_sum = torch.zeros_like(gw)
    for p, (m, s, _) in zip(parts, counted):
        o = sharded.loss_phase(n_global, m, s, p["ids"], p["rewards"], spec.group_size, p["old"], p["ref"], synth.EPS_CLIP,
                               synth.BETA_KL, hidden=p["hidden"], W=batch.W)
        torch.cuda.synchronize()
        loss += o["loss"]
        gw_sum += o["grad_W"]                                                    # the all-reduce's sum
        # a row's log-prob and grad_hidden come out of other tiles than in the unsharded call: equal to rounding
        assert (o["logp"] - lp[p["rows"]]).abs().max().item() <= 1e-5
        scale = gh.float().abs().max().item()
        assert (o["grad_hidden"].float() - gh[p["rows"]].float()).abs().max().item() <= 2.0 ** -7 * scale
    assert torch.allclose(loss, ls, rtol=1e-6, atol=1e-12)
    assert (gw_sum - gw).abs().max().item() <= 2.0 ** -7 * gw.abs().max().item()


def test_fused_step_in_a_group_of_one_against_the_oracle():
    """sharded_grpo_step itself (count phase, loss phase, the three exchanges degenerate in a group of
    one) on the fused LM-head path, every output against the CPU oracle rather than against another
    GPU call."""
    from oracle import rlf_oracle as orc
    spec = synth.scaled(synth.SPECS[3], V=2048 + 136, D=128, w_std=0.3, num_prompts=3, group_size=4, len_lo=20, len_hi=36,
                        spans_lo=1, spans_hi=2, obs_lo=2, obs_hi=4)
    batch = synth.make_batch(spec, DEV)
    out = sharded.sharded_grpo_step(batch.ids, batch.cu_seqlens, batch.rewards, spec.group_size, batch.old_logp,
                                    batch.ref_logp, spec.open_id, spec.close_id, synth.EPS_CLIP, synth.BETA_KL,
                                    hidden=batch.hidden, W=batch.W)
    torch.cuda.synchronize()
    ora = gc.oracle_chain(batch)
    assert np.array_equal(out["mask"].cpu().numpy(), ora["mask"]) and np.array_equal(out["seq_id"].cpu().numpy(), ora["seq_id"])
    assert out["n_local"].item() == out["n_global"].item() == ora["n"]
    assert np.abs(out["adv"].cpu().numpy() - ora["adv64"]).max() <= 1e-6
    r = orc.fused_lmhead_grpo(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W), ora["ids"], ora["seq_id"], ora["adv"],
                              batch.old_logp.cpu().numpy(), batch.ref_logp.cpu().numpy(), ora["mask"], synth.EPS_CLIP,
                              synth.BETA_KL, denom=ora["n"])
    assert np.abs(out["logp"].cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
    from util import loss_close
    lg = out["loss"].cpu().numpy()
    for k in range(3):
        assert loss_close(lg[k], r["loss"][k], gc.loss_floor(ora) if k < 2 else 1e-9, gc.LOSS_RTOL), (k, lg, r["loss"])
    for name in ("grad_hidden", "grad_W"):
        got = out[name].float().cpu().numpy().astype(np.float64)
        assert np.abs(got - r[name]).max() <= 2.0 ** -7 * np.abs(r[name]).max(), name


def test_live_response_count_and_sequence_mean_step_against_the_oracle():
    """rlf_count_live_responses against a count made on the host (a response that is all tool feedback
    carries no loss; a malformed boundary is clipped and flagged), then the sharded step with the
    sequence-mean aggregation and an upper clip width of its own, in a group of one, against the
    oracle's objective function."""
    from oracle import rlf_oracle as orc
    from util import loss_close
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[2], V=4096, num_prompts=3, group_size=4, len_lo=12, len_hi=70, spans_lo=1,
                        spans_hi=2, cover_lo=0.2, cover_hi=0.5)
    batch = synth.make_batch(spec, DEV)
    ora = gc.oracle_chain(batch)
    cu = batch.cu_seqlens.cpu().numpy()
    mask = torch.from_numpy(ora["mask"].copy()).to(DEV)
    mask[cu[2]:cu[3]] = 0                                    # response 2: nothing but observations
    mask[cu[7]:cu[8]] = 0
    want = sum(1 for i in range(len(cu) - 1) if mask[cu[i]:cu[i + 1]].any().item())
    assert want == len(cu) - 3
    got = b.rlf_count_live_responses(mask, batch.cu_seqlens)
    torch.cuda.synchronize()
    assert got.item() == want
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    bad = batch.cu_seqlens.clone()
    bad[-1] = batch.T + 5
    assert b.rlf_count_live_responses(mask, bad, dev_status=st).item() == want and st.item() == 2
    assert b.rlf_count_live_responses(mask[:0], batch.cu_seqlens[:1]).item() == 0

    out = sharded.sharded_grpo_step(batch.ids, batch.cu_seqlens, batch.rewards, spec.group_size, batch.old_logp,
                                    batch.ref_logp, spec.open_id, spec.close_id, 0.2, 0.02, logits=batch.logits,
                                    aggregation=1, eps_clip_high=0.3)
    torch.cuda.synchronize()
    assert out["n_global"].item() == len(cu) - 1              # every response of the recipe carries loss
    r = orc.grpo_loss_obj(gc.to_np(batch.logits), ora["ids"], ora["seq_id"], ora["adv"], batch.old_logp.cpu().numpy(),
                          batch.ref_logp.cpu().numpy(), ora["mask"], 0.2, 0.3, 0.02, aggregation=1, want_coef=True)
    assert np.abs(out["logp"].cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
    lg = out["loss"].cpu().numpy()
    for k in range(3):
        assert loss_close(lg[k], r["loss"][k], 1e-6, gc.LOSS_RTOL), (k, lg, r["loss"])
    guard = gc.near_clip_bound(r["logp"], batch.old_logp.cpu().numpy(), None, eps=0.2) | \
        gc.near_clip_bound(r["logp"], batch.old_logp.cpu().numpy(), None, eps=0.3)
    ulps = gc.grad_ulps(gc.grad_to_f64(out["grad_logits"])[~guard], r["grad"][~guard], ora["ids"][~guard], r["coef"][~guard])
    assert ulps.max() <= gc.GRAD_ULPS


def test_step_with_its_all_reduces_through_nccl_in_a_group_of_one():
    """The three exchanges of sharded_grpo_step issued through torch.distributed's NCCL backend on CUDA
    tensors (one rank: one GPU is all a test gets), in a child process so that the process group, its
    environment and NCCL's state stay out of this one.  The child checks every output against the CPU
    oracle, including a grad_W accumulated over two micro-batches and reduced once."""
    import json
    import os
    import subprocess
    import sys
    child = os.path.join(os.path.dirname(os.path.abspath(__file__)), "nccl_single_rank_child.py")
    env = dict(os.environ, NCCL_NVLS_ENABLE="0")
    p = subprocess.run([sys.executable, child], capture_output=True, text=True, timeout=600, env=env)
    if p.returncode == 77:
        pytest.skip("the NCCL process group could not be created here: " + p.stdout[-300:])
    assert p.returncode == 0, p.stdout[-2000:] + p.stderr[-4000:]
    line = [l for l in p.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["ok"] and res["backend"] == "nccl" and res["world_size"] == 1
    assert len(res["all_reduce_calls"]) == 5
