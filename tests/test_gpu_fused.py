"""GPU parity of the fused LM-head variant (logits formed on the tensor cores, never stored) against
the fp64 oracle.  Tolerances: |d logp| <= 2e-3, loss relative 1e-4; grad_hidden (bf16) and grad_W
(fp32) are sums over V resp. T of bf16-rounded dZ terms, so they are compared per tensor:
max |g - g*| <= 2^-7 max |g*| and cosine similarity >= 0.9999 per row, plus the invariants that hold
at any size (masked rows of grad_hidden are zero, the columns of grad_W sum to zero over V)."""
import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
import gpu_common as gc
from util import loss_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(params=[1, 0], ids=["pair", "single"])
def form(request):
    """Both forms of the contraction kernel: CTA pairs on 256 x 256 tiles, and one CTA per 128 x 256."""
    b = gc.binding()
    b.tune_lmhead(request.param)
    yield request.param
    b.tune_lmhead(1)


def _run(spec, want_grads=True, accumulate=False):
    b = gc.binding()
    batch = synth.make_batch(spec, DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id, dev_status=st)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size, dev_status=st)
    gw0 = None
    if accumulate:
        gw0 = torch.randn((spec.V, spec.D), device=DEV)
    logp, loss, gh, gw = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp,
                                                 batch.ref_logp, mask, synth.EPS_CLIP, synth.BETA_KL, denom=n,
                                                 want_grad_hidden=want_grads, want_grad_W=want_grads,
                                                 grad_W=None if gw0 is None else gw0.clone(),
                                                 accumulate_grad_W=accumulate, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0, st.item()
    ora = gc.oracle_chain(batch)
    r = orc.fused_lmhead_grpo(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W), batch.ids.cpu().numpy(),
                              ora["seq_id"], ora["adv"], batch.old_logp.cpu().numpy(), batch.ref_logp.cpu().numpy(),
                              ora["mask"], synth.EPS_CLIP, synth.BETA_KL, denom=ora["n"],
                              want_grad_hidden=want_grads, want_grad_W=want_grads)
    assert np.array_equal(mask.cpu().numpy(), ora["mask"])
    assert np.abs(logp.cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
    lg = loss.cpu().numpy()
    for k in range(3):
        assert loss_close(lg[k], r["loss"][k], 1e-6, gc.LOSS_RTOL), (k, lg, r["loss"])
    return batch, ora, r, gh, gw, gw0


def _close_tensor(got, want, name):
    got = got.astype(np.float64)
    scale = np.abs(want).max()
    assert np.abs(got - want).max() <= 2.0 ** -7 * scale, (name, np.abs(got - want).max(), scale)
    num = (got * want).sum(axis=1)
    den = np.sqrt((got * got).sum(axis=1) * (want * want).sum(axis=1))
    nz = den > 1e-30 * max(scale, 1e-300) ** 2
    assert (num[nz] / den[nz]).min() >= 0.9999, name


SMALL = dict(len_lo=20, len_hi=20, spans_lo=1, spans_hi=2, obs_lo=2, obs_hi=4)


@pytest.mark.parametrize("V,D", [(2048, 128), (1032, 64), (4096 + 264, 192)])
def test_fused_forward_small(V, D, form):
    """Forward only: several vocabulary tiles with a ragged last tile, one and several k-slabs,
    a token tile that is not full (T = 320 = 2.5 tiles)."""
    spec = synth.scaled(synth.SPECS[3], V=V, D=D, w_std=0.3, **SMALL)
    _run(spec, want_grads=False)


@pytest.mark.parametrize("V,D", [(2048, 128), (1032, 64), (4096 + 264, 320)])
def test_fused_backward_small(V, D, form):
    spec = synth.scaled(synth.SPECS[3], V=V, D=D, w_std=0.3, **SMALL)
    batch, ora, r, gh, gw, _ = _run(spec)
    _close_tensor(gh.float().cpu().numpy(), r["grad_hidden"], "grad_hidden")
    _close_tensor(gw.cpu().numpy(), r["grad_W"], "grad_W")
    assert not gh[torch.from_numpy(ora["mask"] == 0).to(DEV)].any()
    colsum = gw.double().sum(dim=0).abs().max().item()
    assert colsum <= 1e-3 * np.abs(r["grad_W"]).sum(axis=0).max() + 2.0 ** -7 * np.abs(r["grad_W"]).max()


def test_fused_grad_W_accumulates(form):
    spec = synth.scaled(synth.SPECS[3], V=2048, D=128, w_std=0.3, **SMALL)
    batch, ora, r, gh, gw, gw0 = _run(spec, accumulate=True)
    _close_tensor((gw - gw0).cpu().numpy(), r["grad_W"], "grad_W accumulate")


def test_fused_full_vocabulary_and_hidden_reduced_T():
    """Qwen3-4B head (V = 151936 = 593 x 256 + 128, D = 2560 = 40 k-slabs) at 16 x 8 tokens: every
    vocabulary / hidden tile of the full-size launch, with all outputs compared in full."""
    spec = synth.scaled(synth.SPECS[3], len_lo=8, len_hi=8, spans_lo=1, spans_hi=1, obs_lo=1, obs_hi=2)
    batch, ora, r, gh, gw, _ = _run(spec)
    _close_tensor(gh.float().cpu().numpy(), r["grad_hidden"], "grad_hidden")
    _close_tensor(gw.cpu().numpy(), r["grad_W"], "grad_W")


def test_cfg3_full_size_sampled_rows_and_invariants():
    """The launch configuration the benchmark times (T = 32768, D = 2560, V = 151936): log-probs and
    grad_hidden rows of sampled tokens against the oracle (a token's row depends only on that token
    and the batch's token count); every row's log-prob and the scalar loss against the oracle run on
    fp64 logits of the whole batch; sampled rows of grad_W rebuilt from the oracle's per-row outputs; grad_W also through the invariant that its columns sum to zero over the vocabulary."""
    b = gc.binding()
    spec = synth.SPECS[3]
    batch = synth.make_batch(spec, DEV)
    T = batch.T
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id, dev_status=st)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size, dev_status=st)
    logp, loss, gh, gw = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp,
                                                 batch.ref_logp, mask, synth.EPS_CLIP, synth.BETA_KL, denom=n,
                                                 dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    ora = gc.oracle_chain(batch)
    assert np.array_equal(mask.cpu().numpy(), ora["mask"]) and n.item() == ora["n"]

    rng = np.random.default_rng(3)
    live = np.flatnonzero(ora["mask"])
    rows = np.unique(np.concatenate([[0, T - 1], rng.choice(live, size=30, replace=False),
                                     rng.integers(0, T, size=8)]))
    rt = torch.as_tensor(rows, device=DEV)
    r = orc.fused_lmhead_grpo(synth.bf16_bits(batch.hidden[rt]), synth.bf16_bits(batch.W),
                              batch.ids.cpu().numpy()[rows], ora["seq_id"][rows], ora["adv"],
                              batch.old_logp.cpu().numpy()[rows], batch.ref_logp.cpu().numpy()[rows],
                              ora["mask"][rows], synth.EPS_CLIP, synth.BETA_KL, denom=ora["n"],
                              want_grad_hidden=True, want_grad_W=False)
    assert np.abs(logp[rt].cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
    _close_tensor(gh[rt].float().cpu().numpy(), r["grad_hidden"], "grad_hidden rows")
    assert not gh[~mask.bool()].any()

    # every row's log-prob and the scalar loss against the oracle (fp64 logits from the library's
    # fp64 contraction, then the oracle's loss over all 32768 rows)
    logp_o, loss_o, coef_o = gc.oracle_all_rows_through_fp64_head(batch.hidden, batch.W, ora, batch.old_logp.cpu().numpy(),
                                                                  batch.ref_logp.cpu().numpy(), want_coef=True)
    assert np.abs(logp.cpu().numpy() - logp_o).max() <= gc.LOGP_ATOL
    # rows of grad_W at full size: 16 vocabulary rows that are targets of unmasked tokens (their one-hot term
    # matters), 16 random ones and the last row of the ragged last column tile
    vs = np.unique(np.concatenate([ora["ids"][live][:16], rng.integers(0, spec.V, size=16), [spec.V - 1]]))
    gw_o = gc.oracle_grad_W_rows(batch.hidden, batch.W, batch.ids, logp_o, coef_o, vs)
    _close_tensor(gw[torch.as_tensor(vs, device=DEV)].cpu().numpy(), gw_o, "grad_W rows")
    assert np.abs(gw_o).max() >= 0.05 * gw.abs().max().item()      # the sample reaches the tensor's scale
    assert np.abs(logp_o[rows] - r["logp"]).max() <= 1e-9      # the two oracle routes agree on the sampled rows
    lg = loss.cpu().numpy()
    floor = gc.loss_floor(ora)
    for k in range(3):
        assert loss_close(lg[k], loss_o[k], floor if k < 2 else 1e-9, gc.LOSS_RTOL), (k, lg, loss_o)

    col = gw.double().sum(dim=0).abs().max().item()
    assert col <= 1e-3 * gw.double().abs().sum(dim=0).max().item()

    # the same size without the masked rows: identical loss and gradients, NaN log-probs where masked
    logp2, loss2, gh2, gw2 = b.rlf_fused_lmhead_grpo_obj(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp,
                                                         batch.ref_logp, mask, synth.EPS_CLIP, synth.EPS_CLIP,
                                                         synth.BETA_KL, skip_masked=True, denom=n, dev_status=st)
    # and the forward-only sweep over all rows in one launch
    logp3, loss3, _, _ = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp,
                                                 batch.ref_logp, mask, synth.EPS_CLIP, synth.BETA_KL, denom=n,
                                                 want_grad_hidden=False, want_grad_W=False, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    livem = mask.bool()
    assert torch.equal(gh, gh2) and torch.equal(gw, gw2) and torch.equal(loss, loss2)
    assert torch.equal(logp[livem], logp2[livem]) and torch.isnan(logp2[~livem]).all()
    assert (logp3 - logp).abs().max().item() <= 1e-4
    assert loss_close(loss3[0].item(), loss_o[0], floor, gc.LOSS_RTOL)


def test_cfg4_head_shape_reduced_T():
    """Qwen3-8B head (D = 4096 = 64 k-slabs, V = 151936) at 8 x 8 tokens, all outputs in full."""
    spec = synth.scaled(synth.SPECS[4], len_lo=8, len_hi=8, spans_lo=1, spans_hi=1, obs_lo=1, obs_hi=2)
    batch, ora, r, gh, gw, _ = _run(spec)
    _close_tensor(gh.float().cpu().numpy(), r["grad_hidden"], "grad_hidden")
    _close_tensor(gw.cpu().numpy(), r["grad_W"], "grad_W")


def test_fused_micro_batches_with_global_denominator_accumulate():
    """cfg-4-style processing: one response per call, the batch's token count as denominator, grad_W
    accumulated across calls; the sum must equal the single-call result."""
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[4], len_lo=40, len_hi=40, spans_lo=1, spans_hi=2, obs_lo=3, obs_hi=6, V=4096 + 264,
                        D=256, w_std=0.3)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    full = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                   synth.EPS_CLIP, synth.BETA_KL, denom=n)
    torch.cuda.synchronize()
    gw = torch.zeros_like(full[3])
    total = 0.0
    cu = batch.cu_seqlens.cpu().numpy()
    for i in range(batch.B):
        a, e = int(cu[i]), int(cu[i + 1])
        logp, loss, gh, _ = b.rlf_fused_lmhead_grpo(batch.hidden[a:e], batch.W, batch.ids[a:e], seq[a:e], adv,
                                                    batch.old_logp[a:e], batch.ref_logp[a:e], mask[a:e], synth.EPS_CLIP,
                                                    synth.BETA_KL, denom=n, grad_W=gw, accumulate_grad_W=True)
        torch.cuda.synchronize()
        total += loss[0].item()
        assert torch.equal(logp, full[0][a:e])
        assert (gh.float() - full[2][a:e].float()).abs().max().item() <= 2.0 ** -7 * full[2].float().abs().max().item()
    assert abs(total - full[1][0].item()) <= 1e-9 + 1e-6 * abs(full[1][0].item())
    scale = full[3].abs().max().item()
    assert (gw - full[3]).abs().max().item() <= 2.0 ** -7 * scale


@pytest.mark.parametrize("n_live", [0, 1, 129])
def test_fused_backward_runs_over_live_rows_only(n_live, form):
    """The backward contracts over the rows with a non-zero coefficient only.  No live row at all:
    grad_hidden is zero and grad_W is zero (or untouched when accumulating); one live row / one row
    past a 128-row tile: the gradients equal the oracle's."""
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], V=2048, D=128, w_std=0.3, **SMALL)
    batch = synth.make_batch(spec, DEV)
    T = len(batch.ids)
    assert T > 129
    mask_np = np.zeros(T, dtype=np.uint8)
    mask_np[np.random.default_rng(5).permutation(T)[:n_live]] = 1
    mask = torch.from_numpy(mask_np).to(DEV)
    seq = torch.from_numpy(gc.oracle_chain(batch)["seq_id"]).to(DEV)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    n = torch.tensor([max(n_live, 1)], dtype=torch.int64, device=DEV)
    for accumulate in (False, True):
        gw0 = torch.randn((spec.V, spec.D), device=DEV)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        logp, loss, gh, gw = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp,
                                                     batch.ref_logp, mask, synth.EPS_CLIP, synth.BETA_KL, denom=n,
                                                     grad_W=gw0.clone(), accumulate_grad_W=accumulate, dev_status=st)
        torch.cuda.synchronize()
        assert st.item() == 0
        r = orc.fused_lmhead_grpo(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W), batch.ids.cpu().numpy(),
                                  seq.cpu().numpy(), adv.cpu().numpy().astype(np.float64),
                                  batch.old_logp.cpu().numpy(), batch.ref_logp.cpu().numpy(), mask_np,
                                  synth.EPS_CLIP, synth.BETA_KL, denom=int(n.item()))
        got_w = (gw - gw0) if accumulate else gw
        assert not gh[~mask.bool()].any()
        if n_live == 0:
            assert not got_w.any() and not gh.any()
        elif accumulate:
            # (gw0 + g) - gw0 keeps g only to fp32 rounding of gw0 ~ N(0, 1): absolute comparison
            scale = np.abs(r["grad_W"]).max()
            assert np.abs(got_w.cpu().numpy() - r["grad_W"]).max() <= 2.0 ** -7 * scale + 1e-6
        else:
            _close_tensor(got_w.cpu().numpy(), r["grad_W"], "grad_W")
        if n_live:
            live = np.flatnonzero(mask_np)
            _close_tensor(gh.float().cpu().numpy()[live], r["grad_hidden"][live], "grad_hidden")


def test_fused_malformed_rows_are_neutralised_and_reported():
    """A target id outside the vocabulary or a response index outside [0, B) cannot be seen by the
    host: the row gets weight 0 and a zero gradient, a status bit is set, every other row is
    unaffected, and the denominator still counts the mask as given."""
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], V=2048, D=128, w_std=0.3, **SMALL)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    live = torch.nonzero(mask).flatten().cpu().numpy()
    bad_id_rows, bad_seq_row = live[[3, 40]], live[77]
    ids = batch.ids.clone()
    ids[int(bad_id_rows[0])] = spec.V + 5
    ids[int(bad_id_rows[1])] = -1
    seq2 = seq.clone()
    seq2[int(bad_seq_row)] = adv.shape[0]
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    logp, loss, gh, gw = b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, ids, seq2, adv, batch.old_logp, batch.ref_logp,
                                                 mask, synth.EPS_CLIP, synth.BETA_KL, denom=n, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == (b.DEV_BAD_TARGET | b.DEV_BAD_SEQ)
    bad = np.concatenate([bad_id_rows, [bad_seq_row]])
    assert not gh[torch.as_tensor(bad, device=DEV)].any()
    m2 = mask.cpu().numpy().copy()
    m2[bad] = 0
    ids_ok = batch.ids.cpu().numpy().copy()
    seq_ok = seq.cpu().numpy()
    r = orc.fused_lmhead_grpo(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W), ids_ok, seq_ok,
                              adv.cpu().numpy(), batch.old_logp.cpu().numpy(), batch.ref_logp.cpu().numpy(), m2,
                              synth.EPS_CLIP, synth.BETA_KL, denom=int(n.item()))
    good = np.setdiff1d(np.arange(len(ids_ok)), bad_id_rows)
    assert np.abs(logp.cpu().numpy()[good] - r["logp"][good]).max() <= gc.LOGP_ATOL
    assert loss_close(loss[0].item(), r["loss"][0], 1e-6, gc.LOSS_RTOL)
    _close_tensor(gh.float().cpu().numpy(), r["grad_hidden"], "grad_hidden")
    _close_tensor(gw.cpu().numpy(), r["grad_W"], "grad_W")


def _fused_call(b, batch, mask, seq, adv, n, st):
    return b.rlf_fused_lmhead_grpo(batch.hidden, batch.W, batch.ids, seq, adv, batch.old_logp, batch.ref_logp, mask,
                                   synth.EPS_CLIP, synth.BETA_KL, denom=n, dev_status=st)


@pytest.mark.parametrize("V,D", [(2048, 128), (4096 + 264, 320)])
def test_backward_scratch_forms_agree_and_both_match_the_oracle(V, D, form):
    """The two forms of the backward scratch (exponentials against a per-row reference, applied as a row
    factor by the gradient contractions; exponentials against per-tile maxima, rescaled in place) on the
    same batch: each within the per-tensor tolerance of the oracle, the log-probs within rounding of each
    other, and NOT bit-identical gradients (they round dZ at different places), which shows that the
    switch switches something."""
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], V=V, D=D, w_std=0.3, **SMALL)
    batch = synth.make_batch(spec, DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    ora = gc.oracle_chain(batch)
    r = orc.fused_lmhead_grpo(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W), ora["ids"], ora["seq_id"], ora["adv"],
                              batch.old_logp.cpu().numpy(), batch.ref_logp.cpu().numpy(), ora["mask"], synth.EPS_CLIP,
                              synth.BETA_KL, denom=ora["n"])
    outs = {}
    try:
        for row_ref in (1, 0):
            b.tune_lmhead_backward(row_ref)
            logp, loss, gh, gw = _fused_call(b, batch, mask, seq, adv, n, st)
            torch.cuda.synchronize()
            assert st.item() == 0
            assert np.abs(logp.cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
            _close_tensor(gh.float().cpu().numpy(), r["grad_hidden"], "grad_hidden")
            _close_tensor(gw.cpu().numpy(), r["grad_W"], "grad_W")
            outs[row_ref] = (logp, loss, gh, gw)
    finally:
        b.tune_lmhead_backward(1)
    assert (outs[1][0] - outs[0][0]).abs().max().item() <= 1e-4
    assert not torch.equal(outs[1][3], outs[0][3])


def test_row_reference_gives_way_when_a_target_has_vanishing_probability(form):
    """A row's reference is its target logit plus a constant; it stops being usable when the target's
    log-prob falls below about -78 (the row factor or the stored exponentials would leave the normal
    range of bf16).  One live token is given a target logit ~120 below its row maximum: the chunk must be
    redone with per-tile maxima on the device, which shows as results bit-identical to those of the
    per-tile-maximum form (in a chunk that kept its references they differ), and they match the oracle."""
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[3], V=2048, D=128, w_std=0.3, **SMALL)
    batch = synth.make_batch(spec, DEV)
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size)
    live = torch.nonzero(mask).flatten()
    t = int(live[11].item())
    y = int(batch.ids[t].item())
    other = (y + 7) % 1000                                  # not a marker id, not the target
    h = batch.hidden[t].float()
    W = batch.W.clone()
    W[y] = (-60.0 * h / (h * h).sum()).to(torch.bfloat16)      # z[t, y] ~ -60
    W[other] = (60.0 * h / (h * h).sum()).to(torch.bfloat16)   # z[t, other] ~ +60
    batch.W = W
    z_t = (h.double() @ W.double().t())
    assert (z_t.max() - z_t[y]).item() > 100.0
    lp_t = float(z_t[y] - torch.logsumexp(z_t, 0))           # keep that token's ratio and KL term moderate
    batch.old_logp[t] = lp_t + 0.03
    batch.ref_logp[t] = lp_t - 0.05
    ora = gc.oracle_chain(batch)
    r = orc.fused_lmhead_grpo(synth.bf16_bits(batch.hidden), synth.bf16_bits(batch.W), ora["ids"], ora["seq_id"], ora["adv"],
                              batch.old_logp.cpu().numpy(), batch.ref_logp.cpu().numpy(), ora["mask"], synth.EPS_CLIP,
                              synth.BETA_KL, denom=ora["n"])
    assert r["logp"][t] < -100.0
    outs = {}
    try:
        for row_ref in (1, 0):
            b.tune_lmhead_backward(row_ref)
            st = torch.zeros(1, dtype=torch.int32, device=DEV)
            outs[row_ref] = _fused_call(b, batch, mask, seq, adv, n, st)
            torch.cuda.synchronize()
            assert st.item() == 0
    finally:
        b.tune_lmhead_backward(1)
    logp, loss, gh, gw = outs[1]
    assert np.abs(logp.cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
    _close_tensor(gh.float().cpu().numpy(), r["grad_hidden"], "grad_hidden")
    _close_tensor(gw.cpu().numpy(), r["grad_W"], "grad_W")
    for got, want in zip(outs[1], outs[0]):
        assert torch.equal(got, want)
