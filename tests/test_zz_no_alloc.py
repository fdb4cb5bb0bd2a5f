"""The allocation-free loss entry point (rlf_grpo_logp_loss_fwd_bwd_static) against the ordinary one.

Some users of this library cannot allocate device memory where they call it: a training-loop thread
that must not cause the device-wide stall a cudaMalloc brings, a process whose framework already
owns all device memory, a plug-in without access to its host's allocator.  For them the library
carries its own fixed scratch.  This file checks, through the C ABI, that the variant returns what
the workspace-taking entry point returns, twice in a row on different inputs (the shared scratch
keeps the first call's contents, which must not leak into the second), and that it refuses batches
larger than its scratch.  It is collected last on purpose."""
import pytest
import torch

from paper_2509_06980_b200 import synth
import gpu_common as gc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _both(batch, b):
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, batch.spec.open_id, batch.spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    want = b.rlf_grpo_logp_loss_fwd_bwd(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                        synth.EPS_CLIP, synth.BETA_KL, denom=n)
    T = batch.T
    logp = torch.full((T,), 7.0, dtype=torch.float32, device=DEV)
    loss = torch.full((4,), 7.0, dtype=torch.float64, device=DEV)
    grad = torch.full_like(batch.logits, 7.0)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    torch.cuda.synchronize()
    got = b.rlf_grpo_logp_loss_fwd_bwd_static(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp,
                                              mask, synth.EPS_CLIP, synth.BETA_KL, n, logp, loss, grad, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    return want, got


def test_static_scratch_variant_matches_workspace_variant_on_two_calls_in_a_row():
    b = gc.binding()
    first = synth.make_batch(synth.scaled(synth.SPECS[1], len_lo=40, len_hi=40, spans_lo=1, spans_hi=2,
                                          obs_lo=3, obs_hi=6), DEV)
    second = synth.make_batch(synth.scaled(synth.SPECS[1], seed=5, len_lo=24, len_hi=24, spans_lo=1, spans_hi=1,
                                           obs_lo=2, obs_hi=5, V=32768), DEV)
    third = synth.make_batch(synth.SPECS[0], DEV)          # fp32 logits: the general kernel
    for batch in (first, second, third):
        (w_logp, w_loss, w_grad), (g_logp, g_loss, g_grad) = _both(batch, b)
        # the same kernels run on the same inputs, so the agreement is exact; the parity tolerances
        # of the other tests (2e-3 / 1e-4 relative / 2 bf16 ulps) are therefore met with room to spare
        assert torch.equal(g_logp, w_logp)
        assert torch.equal(g_loss, w_loss)
        assert torch.equal(g_grad, w_grad)
        assert (g_logp - w_logp).abs().max().item() <= gc.LOGP_ATOL


@pytest.mark.parametrize("T", [23807, 23808, 32768, 65536])
def test_static_scratch_variant_takes_every_batch_size_up_to_its_stated_maximum(T):
    """Batches near and at RLF_STATIC_MAX_TOKENS (small vocabulary, so the logits stay a few MB): the
    built-in scratch must be as large as the workspace the ordinary entry point asks for at that size.
    23808 is the first size at which an array holding the token records alone would be too small,
    32768 the token count of the Qwen3-4B-shaped micro-batch."""
    b = gc.binding()
    assert T <= b.STATIC_MAX_TOKENS
    g = torch.Generator(device=DEV).manual_seed(T)
    V, B = 64, 16
    logits = (torch.randn((T, V), generator=g, device=DEV) * 3.0).to(torch.bfloat16)
    ids = torch.randint(0, V, (T,), generator=g, device=DEV, dtype=torch.int32)
    seq = (torch.arange(T, device=DEV, dtype=torch.int64) * B // T).to(torch.int32)
    adv = torch.randn(B, generator=g, device=DEV)
    old = -torch.rand(T, generator=g, device=DEV) * 6.0
    ref = old + 0.1 * torch.randn(T, generator=g, device=DEV)
    mask = (torch.rand(T, generator=g, device=DEV) < 0.6).to(torch.uint8)
    n = mask.sum().to(torch.int64).reshape(1)
    want = b.rlf_grpo_logp_loss_fwd_bwd(logits, ids, seq, adv, old, ref, mask, synth.EPS_CLIP, synth.BETA_KL, denom=n)
    for _ in range(2):
        logp = torch.full((T,), 7.0, dtype=torch.float32, device=DEV)
        loss = torch.full((4,), 7.0, dtype=torch.float64, device=DEV)
        grad = torch.full_like(logits, 7.0)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        b.rlf_grpo_logp_loss_fwd_bwd_static(logits, ids, seq, adv, old, ref, mask, synth.EPS_CLIP, synth.BETA_KL,
                                            n, logp, loss, grad, st)
        torch.cuda.synchronize()
        assert st.item() == 0
        assert torch.equal(logp, want[0]) and torch.equal(loss, want[1]) and torch.equal(grad, want[2])


def test_static_scratch_variant_without_a_denominator_counts_the_mask_itself():
    b = gc.binding()
    batch = synth.make_batch(synth.scaled(synth.SPECS[1], len_lo=16, len_hi=16, spans_lo=1, spans_hi=1,
                                          obs_lo=2, obs_hi=4, V=16384), DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, batch.spec.open_id, batch.spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    outs = []
    for _ in range(2):                                   # the counter in the scratch is zeroed per call
        logp = torch.empty(batch.T, dtype=torch.float32, device=DEV)
        loss = torch.empty(4, dtype=torch.float64, device=DEV)
        b.rlf_grpo_logp_loss_fwd_bwd_static(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                            synth.EPS_CLIP, synth.BETA_KL, None, logp, loss, None)
        torch.cuda.synchronize()
        outs.append(loss.clone())
    want = b.rlf_grpo_logp_loss_fwd_bwd(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                        synth.EPS_CLIP, synth.BETA_KL, denom=n, want_grad=False)[1]
    torch.cuda.synchronize()
    assert torch.equal(outs[0], want) and torch.equal(outs[1], want)


def test_static_scratch_variant_refuses_more_tokens_than_it_holds():
    b = gc.binding()
    T = b.STATIC_MAX_TOKENS + 1
    V = 8
    z = torch.zeros((T, V), dtype=torch.bfloat16, device=DEV)
    i32 = torch.zeros(T, dtype=torch.int32, device=DEV)
    f32 = torch.zeros(T, dtype=torch.float32, device=DEV)
    with pytest.raises(b.RlfError) as e:
        b.rlf_grpo_logp_loss_fwd_bwd_static(z, i32, i32, torch.zeros(1, device=DEV), f32, f32,
                                            torch.ones(T, dtype=torch.uint8, device=DEV), 0.2, 0.001, None,
                                            torch.empty(T, device=DEV), torch.empty(4, dtype=torch.float64, device=DEV))
    assert e.value.code == -9
