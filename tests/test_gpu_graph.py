"""The calls queue work on the caller's stream, never synchronise and allocate nothing once their
buffers are given, so a whole step (mask -> advantage -> loss forward + backward; or the fused
LM-head call) can be recorded into a CUDA graph and replayed: the replay must reproduce the eager
results bit for bit, also after the inputs in the captured buffers have been replaced."""
import pytest
import torch

from paper_2509_06980_b200 import synth
import gpu_common as gc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _buffers(b, batch, spec, fused):
    T = batch.T
    B = batch.rewards.shape[0]
    d = dict(mask=torch.empty(T, dtype=torch.uint8, device=DEV), seq=torch.empty(T, dtype=torch.int32, device=DEV),
             n=torch.empty(1, dtype=torch.int64, device=DEV), adv=torch.empty(B, dtype=torch.float32, device=DEV),
             logp=torch.empty(T, dtype=torch.float32, device=DEV), loss=torch.empty(4, dtype=torch.float64, device=DEV),
             st=torch.zeros(1, dtype=torch.int32, device=DEV))
    if fused:
        d["ws"] = b.new_workspace(b.FN_FUSED_LMHEAD, T, spec.V, spec.D, b.RLF_BF16, DEV)
        d["gh"] = torch.empty((T, spec.D), dtype=torch.bfloat16, device=DEV)
        d["gw"] = torch.empty((spec.V, spec.D), dtype=torch.float32, device=DEV)
    else:
        d["ws"] = b.new_workspace(b.FN_LOGP_LOSS, T, spec.V, 0, b.RLF_BF16 if batch.logits.dtype == torch.bfloat16 else b.RLF_F32, DEV)
        d["grad"] = torch.empty_like(batch.logits)
    return d


def _step(b, batch, spec, o, fused):
    b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id, mask_out=o["mask"], seq_id_out=o["seq"],
                          n_out=o["n"], dev_status=o["st"])
    b.rlf_group_advantage(batch.rewards, group_size=spec.group_size, adv_out=o["adv"], dev_status=o["st"])
    if fused:
        b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, o["seq"], o["adv"], batch.old_logp, batch.ref_logp,
                                o["mask"], synth.EPS_CLIP, synth.BETA_KL, denom=o["n"], grad_hidden=o["gh"], grad_W=o["gw"],
                                logp_out=o["logp"], loss_out=o["loss"], workspace=o["ws"], dev_status=o["st"])
    else:
        b.rlf_grpo_logp_loss_fwd_bwd(batch.logits, batch.ids, o["seq"], o["adv"], batch.old_logp, batch.ref_logp, o["mask"],
                                     synth.EPS_CLIP, synth.BETA_KL, denom=o["n"], grad_logits=o["grad"], logp_out=o["logp"],
                                     loss_out=o["loss"], workspace=o["ws"], dev_status=o["st"])


@pytest.mark.parametrize("case", ["cfg0_f32", "bf16_cluster", "fused"])
def test_step_replays_from_a_cuda_graph(case):
    b = gc.binding()
    fused = case == "fused"
    if case == "cfg0_f32":
        spec = synth.SPECS[0]
    elif case == "bf16_cluster":
        spec = synth.scaled(synth.SPECS[1], len_lo=24, len_hi=24, spans_lo=1, spans_hi=1, obs_lo=2, obs_hi=4)
    else:
        spec = synth.scaled(synth.SPECS[3], V=4096 + 264, D=192, w_std=0.3, len_lo=24, len_hi=24, spans_lo=1, spans_hi=2,
                            obs_lo=2, obs_hi=4)
    batch = synth.make_batch(spec, DEV)
    other = synth.make_batch(synth.scaled(spec, seed=spec.seed + 7), DEV)       # same sizes, other contents
    assert other.T == batch.T
    keys = ["mask", "seq", "n", "adv", "logp", "loss"] + (["gh", "gw"] if fused else ["grad"])

    eager = _buffers(b, batch, spec, fused)
    _step(b, batch, spec, eager, fused)                       # also the first call on this device: one-time set-up
    torch.cuda.synchronize()
    want_a = {k: eager[k].clone() for k in keys}
    _step(b, other, spec, eager, fused)
    torch.cuda.synchronize()
    want_b = {k: eager[k].clone() for k in keys}
    assert eager["st"].item() == 0

    o = _buffers(b, batch, spec, fused)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        _step(b, batch, spec, o, fused)                       # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        _step(b, batch, spec, o, fused)
    for k in keys:
        o[k].zero_()
    g.replay()
    torch.cuda.synchronize()
    for k in keys:
        assert torch.equal(o[k], want_a[k]), k
    # new inputs in the captured buffers, same graph
    for name in ("ids", "rewards", "old_logp", "ref_logp") + (("hidden", "W") if fused else ("logits",)):
        getattr(batch, name).copy_(getattr(other, name))
    assert torch.equal(batch.cu_seqlens, other.cu_seqlens)
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    for k in keys:
        assert torch.equal(o[k], want_b[k]), k
    assert o["st"].item() == 0
