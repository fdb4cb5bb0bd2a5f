"""Shared pieces of the GPU parity tests: run one step through the C-ABI binding and through the
oracle on the same bytes, and compare with the stated tolerances."""
import numpy as np
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
from util import loss_close, ulp_error_bf16

LOGP_ATOL = 2e-3          # per-token log-prob, absolute
LOSS_RTOL = 1e-4          # scalar loss, relative
GRAD_ULPS = 2.0           # grad_logits, bf16 ulps of the oracle value
CLIP_GUARD = 1e-4         # rows whose ratio sits this close to a clip bound are not compared element-wise


def binding():
    from paper_2509_06980_b200 import binding as b
    return b


def to_np(t):
    return synth.as_oracle_array(t)


def oracle_chain(batch, logits_np=None, want_grad=True, rows=None):
    """mask -> advantage -> loss on the CPU.  `rows` restricts the loss to a subset of rows (the
    denominator stays the whole batch's)."""
    ids = batch.ids.cpu().numpy()
    cu = batch.cu_seqlens.cpu().numpy()
    mask, seq, n = orc.build_loss_mask(ids, cu, batch.spec.open_id, batch.spec.close_id)
    adv64 = orc.group_advantage(batch.rewards.cpu().numpy(), group_size=batch.tokens.group_size, eps=1e-6)
    adv = adv64.astype(np.float32)
    out = dict(mask=mask, seq_id=seq, n=n, adv64=adv64, adv=adv, ids=ids)
    if logits_np is None:
        return out
    old = batch.old_logp.cpu().numpy()
    ref = batch.ref_logp.cpu().numpy()
    if rows is None:
        r = orc.grpo_loss(logits_np, ids, seq, adv, old, ref, mask, synth.EPS_CLIP, synth.BETA_KL,
                          denom=n, want_grad=want_grad, want_coef=True)
    else:
        r = orc.grpo_loss(logits_np[rows], ids[rows], seq[rows], adv, old[rows], ref[rows], mask[rows],
                          synth.EPS_CLIP, synth.BETA_KL, denom=n, want_grad=want_grad, want_coef=True)
    out.update(r)
    return out


def oracle_all_rows_through_fp64_head(hidden, W, ora, old, ref, row_chunk=2048, want_coef=False):
    """Every row's log-prob and the scalar loss of the fused path from the oracle at full size.
    The head contraction z = H W^T is the one library step: torch.matmul in fp64 on the GPU (bf16
    inputs widened exactly), a chunk of rows at a time; each chunk's fp64 logits go to the host and
    through orc_grpo_loss (dtype f64) with the batch's token count as denominator, so the chunks'
    loss terms add up to the batch's.  Nothing of the library under test is involved.
    -> (logp f64[T], loss f64[4]); with want_coef also the oracle's gradient coefficient c_t of every
    row (grad_z[t, v] = c_t (p[t, v] - [v = y_t]))."""
    T = hidden.shape[0]
    W64 = W.double()
    logp = np.empty(T, np.float64)
    coef = np.empty(T, np.float64)
    loss = np.zeros(4, np.float64)
    for r0 in range(0, T, row_chunk):
        sl = slice(r0, min(T, r0 + row_chunk))
        z = torch.matmul(hidden[sl].double(), W64.t()).cpu().numpy()
        r = orc.grpo_loss(z, ora["ids"][sl], ora["seq_id"][sl], ora["adv"], old[sl], ref[sl], ora["mask"][sl],
                          synth.EPS_CLIP, synth.BETA_KL, denom=ora["n"], want_grad=False, want_coef=want_coef)
        logp[sl] = r["logp"]
        if want_coef:
            coef[sl] = r["coef"]
        loss += np.asarray(r["loss"], np.float64)
        del z
    del W64
    torch.cuda.empty_cache()
    return (logp, loss, coef) if want_coef else (logp, loss)


def oracle_grad_W_rows(hidden, W, ids, logp_o, coef_o, vocab_rows, row_chunk=8192):
    """Rows `vocab_rows` of grad_W at full size from the oracle's per-row outputs and the definition
    grad_W[v, :] = sum_t c_t (p[t, v] - [v = y_t]) hidden[t, :], p[t, v] = exp(z[t, v] - lse_t), with
    lse_t = z[t, y_t] - logp_t.  c_t and logp_t are the oracle's (fp64 logits route); the contractions
    with hidden / W are the library's fp64 matmul on the GPU, a chunk of tokens at a time.
    -> f64 [len(vocab_rows), D]"""
    dev = hidden.device
    vs = torch.as_tensor(np.asarray(vocab_rows), device=dev, dtype=torch.long)
    Wv = W[vs].double()
    T, D = hidden.shape
    out = torch.zeros((len(vocab_rows), D), dtype=torch.float64, device=dev)
    lp = torch.from_numpy(np.asarray(logp_o)).to(dev)
    cf = torch.from_numpy(np.asarray(coef_o)).to(dev)
    y = ids.to(device=dev, dtype=torch.long)
    for r0 in range(0, T, row_chunk):
        sl = slice(r0, min(T, r0 + row_chunk))
        H = hidden[sl].double()
        zy = (H * W[y[sl]].double()).sum(dim=1)
        lse = zy - lp[sl]
        p = torch.exp(H @ Wv.t() - lse[:, None])                   # [rows, len(vs)]
        dz = cf[sl, None] * (p - (y[sl, None] == vs[None, :]).double())
        out += dz.t() @ H
    return out.cpu().numpy()


def loss_floor(ora):
    """Scale below which a relative loss error is not meaningful: the surrogate's mean nearly cancels
    under zero-mean advantages and ratios near one, while a log-prob error e (allowed up to
    LOGP_ATOL) moves a token's term by |A| rho e.  The floor is that permitted movement,
    LOGP_ATOL x mean |A| over the unmasked tokens."""
    a_tok = np.abs(ora["adv"].astype(np.float64))[ora["seq_id"]]
    m = ora["mask"].astype(np.float64)
    return LOGP_ATOL * float((a_tok * m).sum() / max(m.sum(), 1.0))


def gpu_chain(batch, logits, in_place=False, want_grad=True, dev_status=None):
    b = binding()
    mask, seq, n = b.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, batch.spec.open_id, batch.spec.close_id,
                                         dev_status=dev_status)
    adv = b.rlf_group_advantage(batch.rewards, group_size=batch.tokens.group_size, eps=1e-6,
                                dev_status=dev_status)
    logp, loss, grad = b.rlf_grpo_logp_loss_fwd_bwd(logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp,
                                                    mask, synth.EPS_CLIP, synth.BETA_KL, denom=n,
                                                    want_grad=want_grad, in_place=in_place,
                                                    dev_status=dev_status)
    torch.cuda.synchronize()
    return dict(mask=mask, seq_id=seq, n=n, adv=adv, logp=logp, loss=loss, grad=grad)


def near_clip_bound(logp64, old, adv_tok, eps=synth.EPS_CLIP, guard=CLIP_GUARD):
    rho = np.exp(logp64 - old.astype(np.float64))
    return (np.abs(rho - (1 + eps)) < guard) | (np.abs(rho - (1 - eps)) < guard)


def grad_ulps(g, want, ids, coef):
    """Error of grad_logits in bf16 ulps of the oracle value, the target column included: the kernels
    form it as -c S'/S with S' summed over the other columns, which keeps its relative accuracy when
    p_y rounds to one.  The oracle is the definition c (p_y - 1) in fp64 with p_y = exp(z_y - lse): the
    difference is exact only to the rounding of lse, whose sum the oracle takes term after term (up to
    V 2^-53 relative, V <= 2^18), so 2^-35 |c| is taken off the target column's error before it is
    counted in ulps."""
    err = np.abs(np.asarray(g, np.float64) - want)
    t = np.arange(len(ids))
    err[t, ids] = np.maximum(err[t, ids] - 2.0 ** -35 * np.abs(coef), 0.0)
    from util import bf16_ulp
    ulps = err / bf16_ulp(want)
    tiny = (np.abs(want) < 2.0 ** -126) & (np.abs(g) < 2.0 ** -126)
    return np.where(tiny, 0.0, ulps)


def grad_to_f64(g):
    if g.dtype == torch.bfloat16:
        return g.float().cpu().numpy().astype(np.float64)
    return g.cpu().numpy().astype(np.float64)


def check_step(gpu, ora, old_np, grad_rows=None, fp32_grad=False):
    """Compare every output of one step.  grad_rows: row indices of gpu['grad'] that correspond to
    ora['grad'] rows (None = all rows)."""
    assert np.array_equal(gpu["mask"].cpu().numpy(), ora["mask"])
    assert np.array_equal(gpu["seq_id"].cpu().numpy(), ora["seq_id"])
    assert int(gpu["n"].item()) == ora["n"]
    a_gpu = gpu["adv"].cpu().numpy()
    assert np.all(np.abs(a_gpu.astype(np.float64) - ora["adv64"]) <= 1.2e-7 * np.abs(ora["adv64"]) + 1e-30)
    assert np.array_equal(a_gpu == 0, ora["adv64"] == 0)

    logp_gpu = gpu["logp"].cpu().numpy().astype(np.float64)
    rows = np.arange(len(logp_gpu)) if grad_rows is None else np.asarray(grad_rows)
    logp_cmp = logp_gpu if len(ora["logp"]) == len(logp_gpu) else logp_gpu[rows]
    assert np.abs(logp_cmp - ora["logp"]).max() <= LOGP_ATOL

    if len(ora["logp"]) == len(logp_gpu):
        loss_gpu = gpu["loss"].cpu().numpy()
        floor = 1e-6
        for k in range(3):
            assert loss_close(loss_gpu[k], ora["loss"][k], floor, LOSS_RTOL), (k, loss_gpu, ora["loss"])
        assert abs(loss_gpu[3] - ora["loss"][3]) <= 2.0 / max(ora["n"], 1)

    if ora.get("grad") is not None and gpu["grad"] is not None:
        g = grad_to_f64(gpu["grad"][torch.as_tensor(rows, device=gpu["grad"].device)])
        want = ora["grad"]
        seq = ora["seq_id"][rows]
        guard = near_clip_bound(ora["logp"] if len(ora["logp"]) == len(rows) else ora["logp"][rows],
                                old_np[rows], None)
        keep = ~guard
        masked = ora["mask"][rows] == 0
        assert (g[masked] == 0).all(), "masked rows must be exactly zero"
        if fp32_grad:
            err = np.abs(g[keep] - want[keep])
            assert (err <= 1e-4 * np.abs(want[keep]) + 1e-12).all()
        ids_rows = ora["ids"][rows]
        coef_rows = ora["coef"] if len(ora["coef"]) == len(rows) else ora["coef"][rows]
        ulps = grad_ulps(g[keep], want[keep], ids_rows[keep], coef_rows[keep])
        assert ulps.max() <= GRAD_ULPS, ulps.max()
        return float(ulps.max())
    return 0.0
