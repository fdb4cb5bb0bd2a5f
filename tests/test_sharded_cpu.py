"""The sharded single-batch step on CPU: the host-side plan, and the three-exchange step run as two
gloo ranks whose kernels are stood in for by the oracle (tests/oracle_ops.py).  What is checked is
the step logic: the global token count reaches every rank before its loss phase, the ranks' loss
scalars and weight gradients add up to the unsharded result, row gradients stay with their rank."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HERE = os.path.dirname(os.path.abspath(__file__))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_plan_keeps_groups_whole_covers_everything_and_balances():
    from paper_2509_06980_b200 import sharded
    rng = np.random.default_rng(0)
    for world in (1, 2, 3, 8):
        for G in (1, 4, 8):
            n_groups = int(rng.integers(world, 5 * world + 1))
            lens = rng.integers(1, 500, size=n_groups * G)
            cu = np.concatenate([[0], np.cumsum(lens)])
            plan = sharded.plan_shards(cu, G, world)
            assert len(plan) == world
            allr = np.concatenate(plan)
            assert sorted(allr.tolist()) == list(range(n_groups * G))           # each response exactly once
            for p in plan:
                assert (np.diff(p) > 0).all()                                     # batch order kept
                assert (p.reshape(-1, G)[:, 0] % G == 0).all() and (np.diff(p.reshape(-1, G), axis=1) == 1).all()
            gtok = lens.reshape(n_groups, G).sum(axis=1)
            load = [int(lens[p].sum()) for p in plan]
            assert max(load) - min(load) <= gtok.max()                            # greedy bound
    with pytest.raises(ValueError):
        sharded.plan_shards([0, 3, 5, 9], 2, 2)
    # more ranks than groups: the extra ranks get nothing
    plan = sharded.plan_shards([0, 3, 5], 2, 3)
    assert [len(p) for p in plan] == [2, 0, 0]


def test_take_shard_cuts_tokens_and_responses():
    from paper_2509_06980_b200 import sharded
    cu = np.array([0, 3, 5, 9, 10])
    tok = {"ids": np.arange(10), "x": np.arange(10) * 2.0}
    rsp = {"rewards": np.array([0.1, 0.2, 0.3, 0.4])}
    new_cu, t, r = sharded.take_shard(np.array([0, 2]), cu, tok, rsp)
    assert new_cu.tolist() == [0, 3, 7]
    assert t["ids"].tolist() == [0, 1, 2, 5, 6, 7, 8] and r["rewards"].tolist() == [0.1, 0.3]
    new_cu, t, r = sharded.take_shard(np.array([], dtype=np.int64), cu, tok, rsp)
    assert new_cu.tolist() == [0] and len(t["ids"]) == 0 and len(r["rewards"]) == 0


def _problem():
    """4 groups of 2 responses with ragged lengths and observation spans; V = 24, D = 8."""
    rng = np.random.default_rng(11)
    G, V, D = 2, 24, 8
    open_id, close_id = 22, 23
    lens = rng.integers(6, 15, size=8)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    ids = rng.integers(0, 22, size=T).astype(np.int32)
    for b in range(8):
        a = cu[b] + 2
        ids[a], ids[a + 2] = open_id, close_id
    H = torch.from_numpy(rng.normal(size=(T, D)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy((rng.normal(size=(V, D)) * 0.5).astype(np.float32)).to(torch.bfloat16)
    logits = (H.double() @ W.double().t()).float()
    rewards = rng.random(8).astype(np.float32)
    old = rng.normal(-3.0, 0.3, size=T).astype(np.float32)
    ref = rng.normal(-3.0, 0.3, size=T).astype(np.float32)
    return dict(G=G, V=V, D=D, open_id=open_id, close_id=close_id, cu=cu, ids=ids, H=H, W=W, logits=logits,
                rewards=rewards, old=old, ref=ref)


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, HERE)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle_ops
    from paper_2509_06980_b200 import sharded
    P = _problem()
    plan = sharded.plan_shards(P["cu"], P["G"], world)
    tok = {"ids": P["ids"], "old": P["old"], "ref": P["ref"], "rows": np.arange(len(P["ids"]))}
    cu, t, r = sharded.take_shard(plan[rank], P["cu"], tok, {"rewards": P["rewards"]})
    rows = torch.from_numpy(t["rows"])
    common = dict(group_size=P["G"], open_id=P["open_id"], close_id=P["close_id"], eps_clip=0.2, beta_kl=0.05,
                  group=dist.group.WORLD, ops=oracle_ops)
    args = (torch.from_numpy(t["ids"]), torch.from_numpy(cu), torch.from_numpy(r["rewards"]))
    a = sharded.sharded_grpo_step(*args, old_logp=torch.from_numpy(t["old"]), ref_logp=torch.from_numpy(t["ref"]),
                                  logits=P["logits"][rows], **common)
    b = sharded.sharded_grpo_step(*args, old_logp=torch.from_numpy(t["old"]), ref_logp=torch.from_numpy(t["ref"]),
                                  hidden=P["H"][rows], W=P["W"], **common)
    # two micro-batches with accumulation: reduce on the last one only
    half = len(plan[rank]) // 2 // P["G"] * P["G"]
    gw = torch.zeros((P["V"], P["D"]), dtype=torch.float64)
    parts = [plan[rank][:half], plan[rank][half:]]
    n_all = a["n_global"]
    for k, part in enumerate(parts):
        cu_k, t_k, r_k = sharded.take_shard(part, P["cu"], tok, {"rewards": P["rewards"]})
        rows_k = torch.from_numpy(t_k["rows"])
        m, s, _ = sharded.count_phase(torch.from_numpy(t_k["ids"]), torch.from_numpy(cu_k), P["open_id"], P["close_id"],
                                      ops=oracle_ops)
        sharded.loss_phase(n_all, m, s, torch.from_numpy(t_k["ids"]), torch.from_numpy(r_k["rewards"]), P["G"],
                           torch.from_numpy(t_k["old"]), torch.from_numpy(t_k["ref"]), 0.2, 0.05, hidden=P["H"][rows_k],
                           W=P["W"], grad_W=gw, accumulate_grad_W=k > 0, ops=oracle_ops)
    dist.all_reduce(gw)
    # the same two micro-batches through the step itself: accumulate without reducing, then accumulate
    # and reduce once; the batch's token count is handed in, so no count exchange takes place
    gw2 = torch.zeros((P["V"], P["D"]), dtype=torch.float64)
    loss2 = torch.zeros(4, dtype=torch.float64)
    for k, part in enumerate(parts):
        cu_k, t_k, r_k = sharded.take_shard(part, P["cu"], tok, {"rewards": P["rewards"]})
        rows_k = torch.from_numpy(t_k["rows"])
        o = sharded.sharded_grpo_step(torch.from_numpy(t_k["ids"]), torch.from_numpy(cu_k),
                                      torch.from_numpy(r_k["rewards"]), old_logp=torch.from_numpy(t_k["old"]),
                                      ref_logp=torch.from_numpy(t_k["ref"]), hidden=P["H"][rows_k], W=P["W"],
                                      grad_W=gw2, accumulate_grad_W=k > 0, reduce_grad_W=(k == len(parts) - 1),
                                      n_global=n_all, **common)
        assert o["grad_W"] is gw2 and o["n_global"] is n_all
        loss2 += o["loss"]
    # sequence-mean aggregation with an upper clip width of its own: the exchanged count is of responses
    sm = sharded.sharded_grpo_step(*args, old_logp=torch.from_numpy(t["old"]), ref_logp=torch.from_numpy(t["ref"]),
                                   logits=P["logits"][rows], aggregation=1, eps_clip_high=0.3, **common)
    out.put((rank, t["rows"], a["n_local"].item(), a["n_global"].item(), a["loss"].numpy(), a["grad_logits"].numpy(),
             a["logp"].numpy(), b["loss"].numpy(), b["grad_hidden"].numpy(), b["grad_W"].numpy(), gw.numpy(),
             gw2.numpy(), loss2.numpy(), sm["loss"].numpy(), sm["grad_logits"].numpy(), sm["n_local"].item(),
             sm["n_global"].item()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_add_up_to_the_unsharded_step():
    sys.path.insert(0, HERE)
    import oracle_ops
    from paper_2509_06980_b200 import sharded
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = [out.get() for _ in range(2)]
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    got.sort(key=lambda g: g[0])
    # the unsharded step, same stand-in kernels, no process group
    P = _problem()
    common = dict(group_size=P["G"], open_id=P["open_id"], close_id=P["close_id"], eps_clip=0.2, beta_kl=0.05,
                  ops=oracle_ops)
    args = (torch.from_numpy(P["ids"]), torch.from_numpy(P["cu"]), torch.from_numpy(P["rewards"]))
    kw = dict(old_logp=torch.from_numpy(P["old"]), ref_logp=torch.from_numpy(P["ref"]))
    A = sharded.sharded_grpo_step(*args, logits=P["logits"], **kw, **common)
    Bf = sharded.sharded_grpo_step(*args, hidden=P["H"], W=P["W"], **kw, **common)
    S = sharded.sharded_grpo_step(*args, logits=P["logits"], aggregation=1, eps_clip_high=0.3, **kw, **common)
    assert S["n_global"].item() == 8 and not np.allclose(S["loss"].numpy(), A["loss"].numpy())
    n = A["n_global"].item()
    assert got[0][2] + got[1][2] == n and got[0][3] == got[1][3] == n and 0 < got[0][2] < n
    for g in got:
        rows = g[1]
        assert np.allclose(g[4], A["loss"].numpy(), rtol=1e-12, atol=1e-15)          # every rank holds the global loss
        assert np.allclose(g[5], A["grad_logits"].numpy()[rows], rtol=1e-12, atol=1e-18)
        assert np.allclose(g[6], A["logp"].numpy()[rows], rtol=0, atol=1e-13)
        assert np.allclose(g[7], Bf["loss"].numpy(), rtol=1e-12, atol=1e-15)
        assert np.allclose(g[8], Bf["grad_hidden"].numpy()[rows], rtol=1e-11, atol=1e-16)
        assert np.allclose(g[9], Bf["grad_W"].numpy(), rtol=1e-10, atol=1e-15)         # all-reduced weight gradient
        assert np.allclose(g[10], Bf["grad_W"].numpy(), rtol=1e-10, atol=1e-15)        # accumulated, reduced once
        assert np.allclose(g[11], Bf["grad_W"].numpy(), rtol=1e-10, atol=1e-15)        # ... by the step's own flags
        assert np.allclose(g[12], Bf["loss"].numpy(), rtol=1e-12, atol=1e-15)          # micro-batch losses add up
        assert np.allclose(g[13], S["loss"].numpy(), rtol=1e-12, atol=1e-15)           # sequence mean: global loss
        assert np.allclose(g[14], S["grad_logits"].numpy()[rows], rtol=1e-12, atol=1e-18)
        assert g[15] == 4 and g[16] == 8                                              # responses: mine, everyone's
    assert sorted(np.concatenate([got[0][1], got[1][1]]).tolist()) == list(range(len(P["ids"])))
