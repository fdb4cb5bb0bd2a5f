"""Full-size parity in the launch configuration the benchmark times: the Qwen3-4B-shaped micro-batch
(32768 x 151936 bf16, out of place).  The scalar loss and every row's log-prob are compared with
the oracle run over all rows; grad_logits is compared element by element on sampled rows (rows are
independent given the batch's token count), plus properties that hold at any size on all rows."""
import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
import gpu_common as gc
from util import loss_close, ulp_error_bf16

pytestmark = pytest.mark.gpu


def test_cfg1_full_size_against_oracle():
    dev = "cuda"
    batch = synth.make_batch(synth.SPECS[1], dev)
    T, V = batch.logits.shape
    assert (T, V) == (32768, 151936)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    gpu = gc.gpu_chain(batch, batch.logits, dev_status=st)
    assert st.item() == 0

    # all rows: log-prob and scalar loss (oracle forward over the whole batch)
    z_np = gc.to_np(batch.logits)
    ora = gc.oracle_chain(batch, z_np, want_grad=False)
    assert np.array_equal(gpu["mask"].cpu().numpy(), ora["mask"]) and gpu["n"].item() == ora["n"]
    assert np.abs(gpu["logp"].cpu().numpy() - ora["logp"]).max() <= gc.LOGP_ATOL
    lg = gpu["loss"].cpu().numpy()
    for k in range(3):
        assert loss_close(lg[k], ora["loss"][k], 1e-6, gc.LOSS_RTOL), (k, lg, ora["loss"])

    # sampled rows: gradient element by element
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([[0, 1, T - 1], rng.integers(0, T, size=93)]))
    sub = gc.oracle_chain(batch, z_np, want_grad=True, rows=rows)
    g = gc.grad_to_f64(gpu["grad"][torch.as_tensor(rows, device=dev)])
    guard = gc.near_clip_bound(sub["logp"], batch.old_logp.cpu().numpy()[rows], None)
    ulps = ulp_error_bf16(g[~guard], sub["grad"][~guard])
    assert ulps.max() <= gc.GRAD_ULPS
    assert (g[ora["mask"][rows] == 0] == 0).all()

    # all rows: masked rows are zero; live rows sum to ~0 (bf16 rounding noise only)
    grad = gpu["grad"]
    m = gpu["mask"].bool()
    coef_scale = np.abs(ora["coef"]).max()
    for r0 in range(0, T, 4096):
        blk = grad[r0:r0 + 4096]
        mb = m[r0:r0 + 4096]
        assert not blk[~mb].any()
        assert blk[mb].float().sum(dim=1).abs().max().item() <= 0.05 * coef_scale


def test_cfg2_ragged_sampled_rows():
    """Ragged varlen packing (64 responses, lengths 256..4096): tokens and masks at full size, logits
    for a sampled subset of rows (parity needs only independent rows and the batch's token count)."""
    dev = "cuda"
    spec = synth.SPECS[2]
    tok = synth.make_tokens(spec)
    T = len(tok.ids)
    b = gc.binding()
    ids = torch.from_numpy(tok.ids).to(dev)
    cu = torch.from_numpy(tok.cu_seqlens).to(dev)
    mask, seq, n = b.rlf_build_loss_mask(ids, cu, spec.open_id, spec.close_id)
    adv = b.rlf_group_advantage(torch.from_numpy(tok.rewards).to(dev), group_size=spec.group_size)
    torch.cuda.synchronize()
    from oracle import rlf_oracle as orc
    m_o, s_o, n_o = orc.build_loss_mask(tok.ids, tok.cu_seqlens, spec.open_id, spec.close_id)
    assert np.array_equal(mask.cpu().numpy(), m_o) and np.array_equal(seq.cpu().numpy(), s_o) and n.item() == n_o
    assert n_o == T - tok.n_span_tokens

    rng = np.random.default_rng(1)
    rows = np.sort(rng.choice(T, size=600, replace=False))
    sub = synth.scaled(spec, seed=77)
    logits = synth.make_logits(sub, len(rows), dev)
    rows_t = torch.as_tensor(rows, device=dev)
    ids_s, seq_s, mask_s = ids[rows_t].contiguous(), seq[rows_t].contiguous(), mask[rows_t].contiguous()
    center = synth.center_logp(logits, ids_s)
    old, ref = synth.perturbed_logps(sub, center)
    logp, loss, grad = b.rlf_grpo_logp_loss_fwd_bwd(logits, ids_s, seq_s, adv, old, ref, mask_s, synth.EPS_CLIP,
                                                    synth.BETA_KL, denom=n, in_place=False)
    torch.cuda.synchronize()
    a_o = orc.group_advantage(tok.rewards, group_size=spec.group_size, eps=1e-6).astype(np.float32)
    r = orc.grpo_loss(gc.to_np(logits), tok.ids[rows], s_o[rows], a_o, old.cpu().numpy(), ref.cpu().numpy(),
                      m_o[rows], synth.EPS_CLIP, synth.BETA_KL, denom=n_o)
    assert np.abs(logp.cpu().numpy() - r["logp"]).max() <= gc.LOGP_ATOL
    assert loss_close(loss[0].item(), r["loss"][0], 1e-9, gc.LOSS_RTOL)
    guard = gc.near_clip_bound(r["logp"], old.cpu().numpy(), None)
    assert ulp_error_bf16(gc.grad_to_f64(grad)[~guard], r["grad"][~guard]).max() <= gc.GRAD_ULPS


def test_cfg2_full_size_in_place_against_oracle():
    """The ragged recipe at its stated size, the way it has to be run there: one launch over all
    ~133k rows (40 GB of bf16 logits) with grad_logits written over the logits.  The oracle's forward
    pass runs over every row before the call (chunk by chunk, while the logits still exist); 640 sampled
    rows, among them the first and last row of several responses, are snapshotted for the element-wise
    gradient comparison."""
    dev = "cuda"
    spec = synth.SPECS[2]
    batch = synth.make_batch(spec, dev)
    T, V = batch.logits.shape
    assert V == 151936 and 100_000 < T < 180_000 and batch.rewards.shape[0] == 64
    ora = gc.oracle_chain(batch)
    old, ref = batch.old_logp.cpu().numpy(), batch.ref_logp.cpu().numpy()

    logp_o = np.empty(T, np.float64)
    loss_o = np.zeros(4, np.float64)
    for r0 in range(0, T, 4096):
        sl = slice(r0, min(T, r0 + 4096))
        r = orc.grpo_loss(gc.to_np(batch.logits[sl]), ora["ids"][sl], ora["seq_id"][sl], ora["adv"], old[sl], ref[sl],
                          ora["mask"][sl], synth.EPS_CLIP, synth.BETA_KL, denom=ora["n"], want_grad=False)
        logp_o[sl] = r["logp"]
        loss_o += np.asarray(r["loss"], np.float64)

    rng = np.random.default_rng(2)
    cu = batch.tokens.cu_seqlens.astype(np.int64)
    edges = np.concatenate([cu[:9], cu[1:9] - 1, [T - 1]])
    rows = np.unique(np.concatenate([edges, rng.choice(T, size=640, replace=False)]))
    rt = torch.as_tensor(rows, device=dev)
    snap = batch.logits[rt].clone()
    sub = orc.grpo_loss(gc.to_np(snap), ora["ids"][rows], ora["seq_id"][rows], ora["adv"], old[rows], ref[rows],
                        ora["mask"][rows], synth.EPS_CLIP, synth.BETA_KL, denom=ora["n"], want_coef=True)

    st = torch.zeros(1, dtype=torch.int32, device=dev)
    ptr = batch.logits.data_ptr()
    gpu = gc.gpu_chain(batch, batch.logits, in_place=True, dev_status=st)
    assert st.item() == 0 and gpu["grad"].data_ptr() == ptr
    assert np.array_equal(gpu["mask"].cpu().numpy(), ora["mask"]) and gpu["n"].item() == ora["n"]
    assert np.array_equal(gpu["seq_id"].cpu().numpy(), ora["seq_id"])
    assert np.abs(gpu["logp"].cpu().numpy() - logp_o).max() <= gc.LOGP_ATOL
    lg = gpu["loss"].cpu().numpy()
    for k in range(3):
        assert loss_close(lg[k], loss_o[k], 1e-6, gc.LOSS_RTOL), (k, lg, loss_o)

    g = gc.grad_to_f64(gpu["grad"][rt])
    guard = gc.near_clip_bound(sub["logp"], old[rows], None)
    ulps = gc.grad_ulps(g[~guard], sub["grad"][~guard], ora["ids"][rows][~guard], sub["coef"][~guard])
    assert ulps.max() <= gc.GRAD_ULPS
    assert (g[ora["mask"][rows] == 0] == 0).all()

    grad = gpu["grad"]
    m = gpu["mask"].bool()
    coef_scale = np.abs(sub["coef"]).max()
    for r0 in range(0, T, 4096):
        blk, mb = grad[r0:r0 + 4096], m[r0:r0 + 4096]
        assert not blk[~mb].any()
        assert blk[mb].float().sum(dim=1).abs().max().item() <= 0.05 * coef_scale


def test_cfg1_full_size_is_bitwise_stable_over_repeated_launches():
    """No race shows up as run-to-run variation: 12 launches of the full-size step (out of place,
    in place on fresh copies of a slice, and the skip-masked variant) give bit-identical outputs."""
    dev = "cuda"
    b = gc.binding()
    batch = synth.make_batch(synth.SPECS[1], dev)
    first = gc.gpu_chain(batch, batch.logits)
    ref_grad = first["grad"].clone()
    for _ in range(8):
        again = gc.gpu_chain(batch, batch.logits)
        assert torch.equal(again["logp"], first["logp"]) and torch.equal(again["loss"], first["loss"])
        assert torch.equal(again["grad"], ref_grad)
    m = first["mask"].bool()
    for _ in range(3):
        sk = b.rlf_grpo_logp_loss_fwd_bwd_skip_masked(batch.logits, batch.ids, first["seq_id"], first["adv"],
                                                      batch.old_logp, batch.ref_logp, first["mask"], synth.EPS_CLIP,
                                                      synth.BETA_KL, denom=first["n"])
        torch.cuda.synchronize()
        assert torch.equal(sk[2], ref_grad) and torch.equal(sk[1], first["loss"])
        assert torch.equal(sk[0][m], first["logp"][m])
