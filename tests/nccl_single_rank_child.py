"""Child process of tests/test_gpu_sharded.py: sharded_grpo_step with its all-reduces issued through
NCCL on CUDA tensors, in a process group of ONE rank (one GPU is all a test gets).  The reductions are
then identities, so every output must still match the CPU oracle; what the run adds over the
group=None tests is that the three exchanges really go through torch.distributed's NCCL backend with
the tensors the step hands them (int64 count, fp64 loss scalars, fp32 grad_W) and in stream order
with the library's kernels.  Prints one JSON line and exits 0 on success."""
import datetime
import json
import os
import socket
import sys

os.environ.setdefault("NCCL_NVLS_ENABLE", "0")
os.environ.setdefault("NCCL_SOCKET_IFNAME", "lo")        # one rank on this host: the loopback interface will do
HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, HERE)
sys.path.insert(0, os.path.dirname(HERE))

import numpy as np
import torch
import torch.distributed as dist

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import sharded, synth
import gpu_common as gc
from util import loss_close


def main():
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    torch.cuda.set_device(0)
    try:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1,
                                timeout=datetime.timedelta(seconds=120), device_id=torch.device("cuda", 0))
    except Exception as e:           # no NCCL on this machine: nothing of the step has run yet
        print("nccl unavailable: %r" % (e,))
        sys.exit(77)
    calls = []
    real = dist.all_reduce

    def counted(t, *a, **k):
        calls.append((str(t.dtype), tuple(t.shape), t.is_cuda))
        return real(t, *a, **k)
    dist.all_reduce = counted
    try:
        # fused LM-head path, two micro-batches accumulated into one grad_W that is reduced once
        spec = synth.scaled(synth.SPECS[3], V=2048 + 136, D=128, w_std=0.3, num_prompts=4, group_size=4, len_lo=20,
                            len_hi=36, spans_lo=1, spans_hi=2, obs_lo=2, obs_hi=4)
        batch = synth.make_batch(spec, "cuda")
        ora = gc.oracle_chain(batch)
        n_all = ora["n"]
        n_global = torch.tensor([n_all], dtype=torch.int64, device="cuda")
        W = batch.W
        grad_W = torch.zeros(W.shape, dtype=torch.float32, device="cuda")
        want_W = np.zeros(W.shape, np.float64)
        cu_all = batch.cu_seqlens.cpu().numpy()
        tok = {"ids": batch.ids.cpu().numpy(), "old": batch.old_logp.cpu().numpy(), "ref": batch.ref_logp.cpu().numpy(),
               "rows": np.arange(batch.T), "seq": ora["seq_id"], "mask": ora["mask"]}
        for i, responses in enumerate((np.arange(0, 8), np.arange(8, 16))):
            cu, t, r = sharded.take_shard(responses, cu_all, tok, {"rewards": batch.rewards.cpu().numpy()})
            rows = torch.from_numpy(t["rows"]).cuda()
            hidden = batch.hidden[rows].contiguous()
            dev = lambda a: torch.from_numpy(a).cuda()
            out = sharded.sharded_grpo_step(dev(t["ids"]), dev(cu), dev(r["rewards"]), spec.group_size, dev(t["old"]),
                                            dev(t["ref"]), spec.open_id, spec.close_id, synth.EPS_CLIP, synth.BETA_KL,
                                            hidden=hidden, W=W, grad_W=grad_W, accumulate_grad_W=True,
                                            group=dist.group.WORLD, reduce_grad_W=(i == 1), n_global=n_global)
            torch.cuda.synchronize()
            # the oracle on this micro-batch's rows with the whole batch's denominator (response ids
            # renumbered from zero, advantages of its own responses)
            seq_local = t["seq"] - t["seq"].min()
            want = orc.fused_lmhead_grpo(synth.bf16_bits(hidden), synth.bf16_bits(W), t["ids"], seq_local,
                                         ora["adv"][responses], t["old"], t["ref"], t["mask"], synth.EPS_CLIP,
                                         synth.BETA_KL, denom=n_all)
            want_W += want["grad_W"]
            assert np.abs(out["logp"].cpu().numpy() - want["logp"]).max() <= gc.LOGP_ATOL
            lg = out["loss"].cpu().numpy()
            for k in range(3):
                assert loss_close(lg[k], want["loss"][k], gc.loss_floor(ora) if k < 2 else 1e-9, gc.LOSS_RTOL), (k, lg, want["loss"])
            gh = out["grad_hidden"].float().cpu().numpy().astype(np.float64)
            assert np.abs(gh - want["grad_hidden"]).max() <= 2.0 ** -7 * np.abs(want["grad_hidden"]).max()
        got_W = grad_W.cpu().numpy().astype(np.float64)
        assert np.abs(got_W - want_W).max() <= 2.0 ** -7 * np.abs(want_W).max()
        fused_calls = list(calls)
        # n_global was given (no count exchange): per micro-batch the loss scalars, and grad_W once
        assert [c[0] for c in fused_calls] == ["torch.float64", "torch.float32", "torch.float64"], fused_calls
        assert all(c[2] for c in fused_calls)

        # logits path with its own count exchange (int64) and the sequence-mean count of responses
        del calls[:]
        spec2 = synth.scaled(synth.SPECS[2], V=4096, num_prompts=3, group_size=4, len_lo=12, len_hi=70, spans_lo=1,
                             spans_hi=2, obs_lo=2, obs_hi=5, logits_dtype="bf16")
        b2 = synth.make_batch(spec2, "cuda")
        o2 = gc.oracle_chain(b2, gc.to_np(b2.logits))
        out = sharded.sharded_grpo_step(b2.ids, b2.cu_seqlens, b2.rewards, spec2.group_size, b2.old_logp, b2.ref_logp,
                                        spec2.open_id, spec2.close_id, synth.EPS_CLIP, synth.BETA_KL,
                                        logits=b2.logits.clone(), group=dist.group.WORLD)
        torch.cuda.synchronize()
        assert out["n_global"].item() == o2["n"]
        assert np.abs(out["logp"].cpu().numpy() - o2["logp"]).max() <= gc.LOGP_ATOL
        lg = out["loss"].cpu().numpy()
        for k in range(3):
            assert loss_close(lg[k], o2["loss"][k], 1e-6, gc.LOSS_RTOL), (k, lg, o2["loss"])
        assert [c[0] for c in calls] == ["torch.int64", "torch.float64"], calls
        print(json.dumps({"ok": True, "backend": dist.get_backend(), "world_size": dist.get_world_size(),
                          "all_reduce_calls": fused_calls + calls}))
    finally:
        dist.all_reduce = real
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
