"""GPU parity of the forward-only log-prob / entropy entry point against the oracle.
Tolerances: |d logp| <= 2e-3 (as everywhere); |d entropy| <= 2e-3 (fp32 sums of p log p over V)."""
import numpy as np
import pytest
import torch

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
import gpu_common as gc

pytestmark = pytest.mark.gpu
DEV = "cuda"
ENT_ATOL = 2e-3


def _ws(b, form, T, V):
    """`stream`: the entry's own workspace size (chunked streaming kernels); `cluster`: only the loss
    workspace, which selects the row-per-cluster kernel."""
    return b.new_workspace(b.FN_LOGP_ENTROPY if form == "stream" else b.FN_LOGP_LOSS, T, V, 0, b.RLF_BF16, DEV)


@pytest.mark.parametrize("V,dtype,std", [(151936, "bf16", 3.0), (151936, "bf16", 0.5), (4096, "bf16", 8.0),
                                          (1001, "bf16", 2.0), (1024, "f32", 2.0), (8, "bf16", 1.0),
                                          (20480, "bf16", 3.0), (20488, "bf16", 3.0), (40968, "bf16", 3.0),
                                          # unit shapes of the streaming form: 4, 5, 6, 8 vectors per thread
                                          (8192, "bf16", 3.0), (50304, "bf16", 3.0), (12288, "bf16", 3.0),
                                          (32000, "bf16", 3.0)])
@pytest.mark.parametrize("form", ["stream", "cluster"])
def test_logp_and_entropy_match_oracle(V, dtype, std, form):
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[1], V=V, logits_dtype=dtype, logits_std=std, len_lo=12, len_hi=12, spans_lo=1,
                        spans_hi=1, obs_lo=2, obs_hi=3)
    tok = synth.make_tokens(spec)
    T = len(tok.ids)
    logits = synth.make_logits(spec, T, DEV)
    ids = torch.from_numpy(tok.ids).to(DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    logp, ent = b.rlf_logp_entropy_fwd(logits, ids, dev_status=st, workspace=_ws(b, form, T, V))
    torch.cuda.synchronize()
    assert st.item() == 0
    lp_o, h_o = orc.logp_entropy(gc.to_np(logits), tok.ids)
    assert np.abs(logp.cpu().numpy() - lp_o).max() <= gc.LOGP_ATOL
    assert np.abs(ent.cpu().numpy() - h_o).max() <= ENT_ATOL


def test_every_launch_shape_and_special_rows():
    b = gc.binding()
    V, T = 151936, 40
    g = torch.Generator(device=DEV).manual_seed(7)
    z = (torch.randn((T, V), generator=g, device=DEV) * 3).to(torch.bfloat16)
    z[0, :] = 1.5                                 # uniform: H = ln V
    z[1, :] = -30.0
    z[1, 77] = 60.0                               # near one-hot: H ~ 0
    z[2, ::2] = float("-inf")                     # half of the vocabulary has probability zero
    z[3, :] = -1e30                               # huge common offset
    ids = torch.randint(0, V, (T,), generator=g, device=DEV).to(torch.int32)
    ids[1] = 77
    ids[2] = 1
    lp_o, h_o = orc.logp_entropy(gc.to_np(z), ids.cpu().numpy())
    assert abs(h_o[0] - np.log(V)) < 1e-9 and h_o[1] < 1e-20
    for shape in ["stream", (0, 0), (8, 256), (8, 512), (4, 512), (2, 1024), (4, 1024)]:
        form = "stream" if shape == "stream" else "cluster"
        if form == "cluster":
            b.tune_logits_kernel(shape[0], shape[1], -1)
        try:
            st = torch.zeros(1, dtype=torch.int32, device=DEV)
            logp, ent = b.rlf_logp_entropy_fwd(z, ids, dev_status=st, workspace=_ws(b, form, T, V))
            torch.cuda.synchronize()
        finally:
            b.tune_logits_kernel(0, 0, -1)
        assert st.item() == 0
        assert np.abs(logp.cpu().numpy() - lp_o).max() <= gc.LOGP_ATOL, shape
        assert np.abs(ent.cpu().numpy() - h_o).max() <= ENT_ATOL, shape


def test_matches_the_training_entry_point_and_flags_bad_targets():
    b = gc.binding()
    spec = synth.scaled(synth.SPECS[1], len_lo=16, len_hi=16, spans_lo=1, spans_hi=1, obs_lo=2, obs_hi=3)
    batch = synth.make_batch(spec, DEV)
    full = gc.gpu_chain(batch, batch.logits, want_grad=False)
    logp, _ = b.rlf_logp_entropy_fwd(batch.logits, batch.ids, want_entropy=False)
    logp_c, _ = b.rlf_logp_entropy_fwd(batch.logits, batch.ids, want_entropy=False,
                                       workspace=_ws(b, "cluster", len(batch.ids), spec.V))
    torch.cuda.synchronize()
    assert (logp - full["logp"]).abs().max().item() <= 1e-5
    assert (logp_c - full["logp"]).abs().max().item() <= 1e-5
    ids = batch.ids.clone()
    ids[3] = spec.V
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    logp2, ent2 = b.rlf_logp_entropy_fwd(batch.logits, ids, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == b.DEV_BAD_TARGET
    assert torch.equal(logp2[4:], logp[4:]) and torch.isnan(logp2[3]) and torch.isfinite(ent2[3])
