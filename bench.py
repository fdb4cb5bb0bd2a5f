#!/usr/bin/env python
"""Benchmark of the GRPO policy-update loss path on B200.

One step = one pass of the whole path over one synthetic micro-batch that is already resident in
HBM:  rlf_build_loss_mask -> rlf_group_advantage -> rlf_grpo_logp_loss_fwd_bwd  (forward and
backward over the full vocabulary).  The workload at one GPU is the Qwen3-4B-shaped micro-batch:
16 responses x 2048 tokens, V = 151936 bf16 logits (9.96 GB in, 9.96 GB of grad_logits out).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line.  With N > 1 (under torchrun) every rank runs its own micro-batch (no data-path
collective: tokens are independent given the per-batch token count), the time is the max over
ranks, and the value is the tokens all ranks processed per second.
`--impl reference` times the fp64 CPU oracle on the host cores instead (a deliberately slow
definition-level program; rank 0 only).
"""
import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2509_06980_b200 import synth

METRIC = "GRPO loss fwd+bwd tokens/s at V=151936 bf16"
UNIT = "tokens/s"
WORKLOAD = "cfg1_qwen3_4b_microbatch: 16 responses x 2048 tokens, V=151936 bf16 logits"

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/.  Each figure is valid only for the source text it was captured from: the key is the
# hash that `python bench.py --source-keys` printed when the capture was taken, and a figure whose key
# no longer matches the tree is reported as null.
#   row kernel: one full-size launch (32768 rows; a one-pass capture), per token;
#   streaming forward kernel: the T = 4096 capture, per token (traffic is proportional to rows);
#   fused LM-head: every kernel of one forward / one forward + backward call at cfg 3 full size
#   (one-pass capture of the whole call), per call.
NCU_TRAFFIC = {"logits_loss_cu_sha1": "ee482c3f18de39e50fed56d917e964b8673b1d59", "dram_bytes_per_token": 606028.0}
NCU_TRAFFIC_FUSED = {"lmhead_cu_sha1": "23538aaabeed8d9a0c763b7f7e3bb6ee625b306d",
                     "fwd_bytes_per_call": 3957591808.0, "fwd_bwd_bytes_per_call": 34875904256.0}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _tensor_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            j = json.load(f)
        return float(j["bf16_tflops"]), float(j["bf16_tflops_sustained"]), "measured"
    return 1590.0, 1400.0, "fallback"


def time_fused_lmhead(rlf, dev, steps, tokens_per_response=0, cfg=3, responses=0):
    """The fused LM-head variant on the Qwen3-4B head (T = 32768, D = 2560, V = 151936): forward
    (log-probs and loss, logits never stored) and forward + backward (grad_hidden, grad_W)."""
    spec = synth.SPECS[cfg]
    if tokens_per_response:
        spec = synth.scaled(spec, len_lo=tokens_per_response, len_hi=tokens_per_response)
    if responses:
        spec = synth.scaled(spec, num_prompts=1, group_size=responses)     # fewer full-length responses
    tok = synth.make_tokens(spec)
    T = len(tok.ids)
    ids = torch.from_numpy(tok.ids).to(dev)
    cu = torch.from_numpy(tok.cu_seqlens).to(dev)
    H, W = synth.make_hidden_and_head(spec, T, dev)
    mask, seq, n = rlf.rlf_build_loss_mask(ids, cu, spec.open_id, spec.close_id)
    adv = rlf.rlf_group_advantage(torch.from_numpy(tok.rewards).to(dev), group_size=spec.group_size)
    center = synth.center_logp_from_head(H, W, ids)
    old, ref = synth.perturbed_logps(spec, center)
    del center
    ws = rlf.new_workspace(rlf.FN_FUSED_LMHEAD, T, spec.V, spec.D, rlf.RLF_BF16, dev)
    gh = torch.empty((T, spec.D), dtype=torch.bfloat16, device=dev)
    gw = torch.empty((spec.V, spec.D), dtype=torch.float32, device=dev)
    logp = torch.empty(T, dtype=torch.float32, device=dev)
    loss = torch.empty(4, dtype=torch.float64, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)

    def run(bwd):
        rlf.rlf_fused_lmhead_grpo(H, W, ids, seq, adv, old, ref, mask, synth.EPS_CLIP, synth.BETA_KL, denom=n,
                                  want_grad_hidden=bwd, want_grad_W=bwd, grad_hidden=gh if bwd else None,
                                  grad_W=gw if bwd else None, logp_out=logp, loss_out=loss, workspace=ws,
                                  dev_status=st)
    out = {"workload": "%s: hidden [%d, %d] x W [151936, %d] bf16" % (spec.name, T, spec.D, spec.D), "T": T, "D": spec.D,
           "V": spec.V}
    burst, sustained, kind = _tensor_peaks()
    # the backward contracts only over the unmasked rows, so its flops are counted over those rows:
    # two GEMMs each (the forward's exponentials are kept for them: nothing is recomputed)
    live = int(mask.sum().item())
    out["live_rows"] = live
    tvd = 2.0 * spec.V * spec.D
    # Tensor-core work is power-bound here: a kernel timed in the first second after an idle spell runs
    # at clocks it cannot hold.  Every variant is therefore looped for warm_s seconds before it is timed
    # (profiling captures at reduced size skip this: they take their figures from the counters).
    full_size = not (tokens_per_response or responses)
    warm_s = 1.5 if full_size else 0.0

    def warm(fn):
        fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < warm_s:
            for _ in range(4):
                fn()
            torch.cuda.synchronize()

    for name, bwd, useful_flops, executed_flops in (("fwd", False, tvd * T, tvd * T),
                                                    ("fwd_bwd", True, tvd * (T + 2 * live), tvd * (T + 2 * live))):
        warm(lambda: run(bwd))
        ts = []
        for _ in range(steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            run(bwd)
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        ms = statistics.mean(ts)
        useful = useful_flops / ms / 1e9
        out[name] = {"ms": ms, "tokens_per_s": T / ms * 1e3, "useful_tflops": useful,
                     "executed_tflops": executed_flops / ms / 1e9,
                     "dense_equivalent_tflops": tvd * T * (3 if bwd else 1) / ms / 1e9,
                     "roofline": {"bound": "tensor", "achieved": useful, "peak": burst, "unit": "TFLOP/s",
                                  "frac": useful / burst, "peak_kind": "of " + kind + " (burst)",
                                  "frac_of_sustained": useful / sustained, "frac_of_nominal_2250": useful / 2250.0,
                                  "traffic": (NCU_TRAFFIC_FUSED["fwd_bwd_bytes_per_call" if bwd else "fwd_bytes_per_call"]
                                              if full_size and cfg == 3 and NCU_TRAFFIC_FUSED["lmhead_cu_sha1"] == _lmhead_sha1()
                                              else None)}}
    # the same call without multiplying the masked rows at all (their log-prob is not produced)
    def run_skip():
        rlf.rlf_fused_lmhead_grpo_obj(H, W, ids, seq, adv, old, ref, mask, synth.EPS_CLIP, synth.EPS_CLIP,
                                      synth.BETA_KL, skip_masked=True, denom=n, grad_hidden=gh, grad_W=gw,
                                      logp_out=logp, loss_out=loss, workspace=ws, dev_status=st)
    warm(run_skip)
    ts = []
    for _ in range(steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        run_skip()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ms = statistics.mean(ts)
    out["fwd_bwd_skip_masked"] = {"entry": "rlf_fused_lmhead_grpo_obj(skip_masked=1)", "ms": ms,
                                  "tokens_per_s": T / ms * 1e3, "executed_tflops": tvd * 3 * live / ms / 1e9}
    if st.item() != 0:
        out["device_status"] = int(st.item())
    out["loss"] = float(loss[0].item())
    # forward-only log-prob + entropy from hidden states (the old / reference policy pass)
    ws_lp = rlf.new_workspace(rlf.FN_FUSED_LOGP_ENTROPY, T, spec.V, spec.D, rlf.RLF_BF16, dev)
    ent = torch.empty(T, dtype=torch.float32, device=dev)
    run_lp = lambda: rlf.rlf_fused_lmhead_logp_entropy(H, W, ids, logp_out=logp, entropy_out=ent, workspace=ws_lp)
    warm(run_lp)
    ts = []
    for _ in range(steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        run_lp()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ms = statistics.mean(ts)
    out["fwd_logp_entropy"] = {"entry": "rlf_fused_lmhead_logp_entropy", "ms": ms, "tokens_per_s": T / ms * 1e3,
                               "executed_tflops": tvd * T / ms / 1e9}
    if not tokens_per_response and not responses:
        # context: the library GEMM of the forward's shape on this GPU, in the same state (back to back,
        # logits written to HBM as bf16): what an unfused path pays for the contraction alone
        z = torch.empty((T, spec.V), dtype=torch.bfloat16, device=dev)
        warm(lambda: torch.matmul(H, W.t(), out=z))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            torch.matmul(H, W.t(), out=z)
        b.record()
        torch.cuda.synchronize()
        lib_ms = a.elapsed_time(b) / steps
        out["library_gemm_same_shape"] = {"what": "torch.matmul(H, W^T) -> bf16 [T, V], not part of the path",
                                          "ms": lib_ms, "tflops": tvd * T / lib_ms / 1e9}
        del z
    return out


# the same for the forward-only log-prob + entropy pass (profiles/logp_entropy_stream_kernel_T4096_ncu_full.md)
NCU_TRAFFIC_ENTROPY = {"section_sha1": "cbd417db69ba91bea4be00d3c9c3cda5dee7abb9", "dram_bytes_per_token": 305813.0}


def _entropy_section_sha1():
    """Hash of the forward-only section of logits_loss.cu (streaming and merge kernels, entry point)."""
    p = os.path.join(ROOT, "paper_2509_06980_b200", "csrc", "logits_loss.cu")
    with open(p, "rb") as f:
        text = f.read()
    a = text.find(b"// Forward-only log-prob (+ entropy) of given target ids")
    b = text.find(b"// Skip-masked variant:")
    return hashlib.sha1(text[a:b] if 0 <= a < b else text).hexdigest()


def _lmhead_sha1():
    """Hash of the fused LM-head source file."""
    with open(os.path.join(ROOT, "paper_2509_06980_b200", "csrc", "lmhead.cu"), "rb") as f:
        return hashlib.sha1(f.read()).hexdigest()


def _kernel_sha1():
    """Hash of the row kernel's source text (from its section header to the general kernel's)."""
    p = os.path.join(ROOT, "paper_2509_06980_b200", "csrc", "logits_loss.cu")
    with open(p, "rb") as f:
        text = f.read()
    a = text.find(b"// Fast row kernel\n")
    b = text.find(b"// General row kernel:")
    return hashlib.sha1(text[a:b] if 0 <= a < b else text).hexdigest()


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            try:
                pw.append(float(c[3]))
            except ValueError:
                pass
            for name, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
            # settled part of the run only (the first third still carries the previous state's clocks)
            tail = sm[len(sm) // 3:]
            out["sm_mhz_settled"] = statistics.median(tail)
            if pw:
                out["power_w_settled"] = statistics.median(pw[len(pw) // 3:])
        return out


def workload_config(world, tokens_per_response=0):
    """The `config` object of the JSON line: the workload alone (the same for the CUDA arm and for the
    oracle arm, which runs bounded samples of it), nothing about how an arm computes."""
    spec = synth.SPECS[1]
    tok = tokens_per_response or spec.len_hi
    B = spec.num_prompts * spec.group_size
    return {"workload": WORKLOAD if not tokens_per_response else "cfg1 recipe at %d tokens per response" % tokens_per_response,
            "T": B * tok, "V": spec.V, "B": B, "G": spec.group_size, "eps_clip": synth.EPS_CLIP, "beta_kl": synth.BETA_KL,
            "parallelism": "independent micro-batch per GPU" if world > 1 else "single GPU"}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def shard_seed(base_seed, rank):
    """Each rank draws its own micro-batch of the same recipe."""
    return base_seed + 101 * rank


def aggregate(tokens_per_rank, world, max_seconds):
    """Whole-job throughput: the tokens all ranks processed over the slowest rank's time."""
    return tokens_per_rank * world / max_seconds


def max_over_ranks(seconds, world, device=None):
    """Slowest rank's time (an all-reduce MAX of one scalar; identity at world size 1)."""
    if world <= 1:
        return float(seconds)
    import torch.distributed as dist
    t = torch.tensor([seconds], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ---------------------------------------------------------------------------------------------
def oracle_step_sampler(batch, rows_per_call):
    """Returns f(k) that runs the oracle's loss forward + backward on the k-th slice of
    `rows_per_call` rows and returns (rows done, seconds the oracle computed).  The mask and the
    advantages of the whole batch are formed once, before any clock starts (5 bytes per token against
    600 KB per token for the loss), and a slice is staged in host memory before its clock starts, so
    the figure is the oracle's arithmetic alone wherever the batch lives."""
    from oracle import rlf_oracle as orc
    ids = batch.ids.cpu().numpy()
    cu = batch.cu_seqlens.cpu().numpy()
    rewards = batch.rewards.cpu().numpy()
    old = batch.old_logp.cpu().numpy()
    ref = batch.ref_logp.cpu().numpy()
    T = batch.T
    mask, seq, n = orc.build_loss_mask(ids, cu, batch.spec.open_id, batch.spec.close_id)
    adv = orc.group_advantage(rewards, group_size=batch.tokens.group_size, eps=1e-6).astype(np.float32)

    def run(k):
        r0 = (k * rows_per_call) % T
        r1 = min(T, r0 + rows_per_call)
        z = np.ascontiguousarray(synth.as_oracle_array(batch.logits[r0:r1]))
        t0 = time.perf_counter()
        orc.grpo_loss(z, ids[r0:r1], seq[r0:r1], adv, old[r0:r1], ref[r0:r1], mask[r0:r1], synth.EPS_CLIP,
                      synth.BETA_KL, denom=n, want_grad=True)
        return r1 - r0, time.perf_counter() - t0
    return run, orc.num_threads()


def time_oracle(batch, budget_s, rows_per_call=256):
    run, cores = oracle_step_sampler(batch, rows_per_call)
    run(0)                                      # page in, build
    done, k, busy = 0, 0, 0.0
    while busy < budget_s and k < 4096:
        rows, sec = run(k)
        done += rows
        busy += sec
        k += 1
    return dict(value=done / busy, unit=UNIT, cores=cores, kind="oracle",
                sample="%d rows of the same micro-batch (full vocabulary, forward + fp64 gradient), %d calls of %d rows, "
                       "%.1f s of oracle time (slices staged in host memory outside the clock)"
                       % (done, k, rows_per_call, busy))


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    spec = synth.SPECS[1]
    rows = 256
    # the oracle reads a row slice per step; draw only what the steps touch
    need = rows * (args.steps + max(args.warmup, 2))
    per = max(need // 16 + 1, 64)
    small = synth.scaled(spec, len_lo=per, len_hi=per, spans_lo=1, spans_hi=2, obs_lo=10, obs_hi=20)
    batch = synth.make_batch(small, "cpu")
    run, cores = oracle_step_sampler(batch, rows)
    for k in range(max(args.warmup, 2)):        # at least two untimed calls: thread start-up, page-in
        run(k)
    done, el = 0, 0.0
    for k in range(args.steps):
        rows_done, sec = run(max(args.warmup, 2) + k)
        done += rows_done
        el += sec
    val = done / el
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * el / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(max(1, args.gpus)),
        "step": "fp64 CPU oracle on %d rows per step (bounded sample of the workload)" % rows,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "%d rows per step x %d steps, full vocabulary, forward + fp64 gradient"
                                   % (rows, args.steps)},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
def run_fused_only(args):
    """Only the fused LM-head variant, optionally at a reduced token count (profiling captures)."""
    from paper_2509_06980_b200 import binding as rlf
    torch.cuda.set_device(0)
    out = time_fused_lmhead(rlf, torch.device("cuda", 0), max(1, args.steps), args.tokens_per_response,
                            cfg=args.fused_cfg, responses=args.responses)
    print(json.dumps({"fused_lmhead": out, "gpu_launches": rlf.launch_count()}))


def run_fused_phases(args):
    """Sustained cost of the fused LM-head call by phase (cfg 3 or 4): each variant is looped for
    --phase-seconds with the SM clock and board power sampled, so that what the power cap costs each
    phase shows.  Variants differ by one phase at a time (forward sweep over the unmasked rows; plus
    grad_hidden; plus grad_W; plus both; plus the masked rows' log-probs).  Prints one JSON line."""
    from paper_2509_06980_b200 import binding as rlf
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    spec = synth.SPECS[args.fused_cfg]
    tok = synth.make_tokens(spec)
    T = len(tok.ids)
    ids = torch.from_numpy(tok.ids).to(dev)
    cu = torch.from_numpy(tok.cu_seqlens).to(dev)
    H, W = synth.make_hidden_and_head(spec, T, dev)
    mask, seq, n = rlf.rlf_build_loss_mask(ids, cu, spec.open_id, spec.close_id)
    adv = rlf.rlf_group_advantage(torch.from_numpy(tok.rewards).to(dev), group_size=spec.group_size)
    center = synth.center_logp_from_head(H, W, ids)
    old, ref = synth.perturbed_logps(spec, center)
    del center
    ws = rlf.new_workspace(rlf.FN_FUSED_LMHEAD, T, spec.V, spec.D, rlf.RLF_BF16, dev)
    gh = torch.empty((T, spec.D), dtype=torch.bfloat16, device=dev)
    gw = torch.empty((spec.V, spec.D), dtype=torch.float32, device=dev)
    logp = torch.empty(T, dtype=torch.float32, device=dev)
    loss = torch.empty(4, dtype=torch.float64, device=dev)
    z = torch.empty((T, spec.V), dtype=torch.bfloat16, device=dev)
    live = int(mask.sum().item())

    def call(skip, want_gh, want_gw):
        rlf.rlf_fused_lmhead_grpo_obj(H, W, ids, seq, adv, old, ref, mask, synth.EPS_CLIP, synth.EPS_CLIP, synth.BETA_KL,
                                      skip_masked=skip, denom=n, want_grad_hidden=want_gh, want_grad_W=want_gw,
                                      grad_hidden=gh if want_gh else None, grad_W=gw if want_gw else None,
                                      logp_out=logp, loss_out=loss, workspace=ws)
    tvd = 2.0 * spec.V * spec.D
    variants = [
        ("library_gemm_all_rows", lambda: torch.matmul(H, W.t(), out=z), tvd * T),
        ("sweep_all_rows", lambda: call(False, False, False), tvd * T),
        ("sweep_unmasked_rows", lambda: call(True, False, False), tvd * live),
        ("sweep_unmasked_plus_grad_hidden", lambda: call(True, True, False), tvd * 2 * live),
        ("sweep_unmasked_plus_grad_W", lambda: call(True, False, True), tvd * 2 * live),
        ("sweep_unmasked_plus_both_gradients", lambda: call(True, True, True), tvd * 3 * live),
        ("full_call_all_log_probs_both_gradients", lambda: call(False, True, True), tvd * (T + 2 * live)),
    ]
    out = {"workload": "%s: hidden [%d, %d] x W [%d, %d] bf16" % (spec.name, T, spec.D, spec.V, spec.D),
           "unmasked_rows": live, "seconds_per_variant": args.phase_seconds, "variants": {}}
    for name, fn, flops in variants:
        fn()
        torch.cuda.synchronize()
        sampler = ClockSampler(0)
        sampler.start()
        t0 = time.perf_counter()
        k = 0
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        while time.perf_counter() - t0 < args.phase_seconds:
            for _ in range(4):
                fn()
            k += 4
            torch.cuda.synchronize()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / k
        clocks = sampler.stop()
        out["variants"][name] = {"ms": ms, "executed_tflops": flops / ms / 1e9, "sm_mhz": clocks.get("sm_mhz_settled"),
                                 "power_w": clocks.get("power_w_settled"), "reasons": clocks["reasons"]}
    print(json.dumps({"fused_phases": out, "gpu_launches": rlf.launch_count()}))


def run_other_configs(args):
    """The configurations that are parity cases rather than the headline: cfg 2 (ragged packing, ~133k
    tokens, logits processed in place) and cfg 4 (8 micro-batches of 8192 tokens with a global
    denominator; logits path and fused LM-head path).  Prints one JSON line."""
    from paper_2509_06980_b200 import binding as rlf
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    steps = max(2, min(args.steps, 5))
    out = {}

    def timed(fn, n):
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(n):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.mean(ts)

    # cfg 0 (tiny, latency-bound): the whole step launched call by call and replayed from a CUDA graph
    spec0 = synth.SPECS[0]
    b0 = synth.make_batch(spec0, dev)
    o = dict(mask=torch.empty(b0.T, dtype=torch.uint8, device=dev), seq=torch.empty(b0.T, dtype=torch.int32, device=dev),
             n=torch.empty(1, dtype=torch.int64, device=dev), adv=torch.empty(b0.rewards.shape[0], device=dev),
             logp=torch.empty(b0.T, device=dev), loss=torch.empty(4, dtype=torch.float64, device=dev),
             grad=torch.empty_like(b0.logits), ws=rlf.new_workspace(rlf.FN_LOGP_LOSS, b0.T, spec0.V, 0, rlf.RLF_F32, dev))

    def step0():
        rlf.rlf_build_loss_mask(b0.ids, b0.cu_seqlens, spec0.open_id, spec0.close_id, mask_out=o["mask"],
                                seq_id_out=o["seq"], n_out=o["n"])
        rlf.rlf_group_advantage(b0.rewards, group_size=spec0.group_size, adv_out=o["adv"])
        rlf.rlf_grpo_logp_loss_fwd_bwd(b0.logits, b0.ids, o["seq"], o["adv"], b0.old_logp, b0.ref_logp, o["mask"],
                                       synth.EPS_CLIP, synth.BETA_KL, denom=o["n"], grad_logits=o["grad"],
                                       logp_out=o["logp"], loss_out=o["loss"], workspace=o["ws"])

    def per_step_us(fn, reps=200):
        for _ in range(10):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / reps
    eager_us = per_step_us(step0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step0()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step0()
    out["cfg0_tiny_step_latency"] = {"T": b0.T, "V": spec0.V, "launches_per_step": 6, "eager_us": eager_us,
                                     "cuda_graph_us": per_step_us(graph.replay)}
    del b0, o, graph

    # the logits path at other vocabulary sizes (not stated configurations; about 4 GB of bf16 logits each,
    # out of place, so 8 GB moved per call), as a fraction of the measured copy rate
    peak_gbs, peak_kind = _peaks()
    vocab = {}
    g = torch.Generator(device=dev)
    g.manual_seed(0)
    for V_other in (32000, 50304, 128256, 200000, 262144):
        Tv = int(4e9 // (2 * V_other)) // 16 * 16
        z = torch.empty((Tv, V_other), dtype=torch.bfloat16, device=dev).normal_(0, 3, generator=g)
        gz = torch.empty_like(z)
        ids_v = torch.randint(0, V_other, (Tv,), device=dev, generator=g).to(torch.int32)
        seq_v = (torch.arange(Tv, device=dev) * 16 // Tv).to(torch.int32)
        adv_v = torch.randn(16, device=dev, generator=g)
        mask_v = (torch.rand(Tv, device=dev, generator=g) < 0.55).to(torch.uint8)
        old_v = torch.full((Tv,), -12.0, device=dev)
        n_v = mask_v.sum().to(torch.int64).reshape(1)
        ws_v = rlf.new_workspace(rlf.FN_LOGP_LOSS, Tv, V_other)
        wse_v = rlf.new_workspace(rlf.FN_LOGP_ENTROPY, Tv, V_other)
        lp_v = torch.empty(Tv, dtype=torch.float32, device=dev)
        ent_v = torch.empty(Tv, dtype=torch.float32, device=dev)
        ls_v = torch.empty(4, dtype=torch.float64, device=dev)
        ms_t = timed(lambda: rlf.rlf_grpo_logp_loss_fwd_bwd(z, ids_v, seq_v, adv_v, old_v, old_v, mask_v, synth.EPS_CLIP,
                                                            synth.BETA_KL, denom=n_v, grad_logits=gz, logp_out=lp_v,
                                                            loss_out=ls_v, workspace=ws_v), 4 * steps)
        ms_f = timed(lambda: rlf.rlf_logp_entropy_fwd(z, ids_v, logp_out=lp_v, entropy_out=ent_v, workspace=wse_v), 4 * steps)
        gbs_t = Tv * V_other * 4 / ms_t / 1e6
        gbs_f = Tv * V_other * 2 / ms_f / 1e6
        vocab[str(V_other)] = {"T": Tv, "fwd_bwd_ms": ms_t, "fwd_bwd_gbs": gbs_t, "fwd_bwd_frac": gbs_t / peak_gbs,
                               "logp_entropy_ms": ms_f, "logp_entropy_gbs": gbs_f, "logp_entropy_frac": gbs_f / peak_gbs}
        del z, gz, ws_v, wse_v
        torch.cuda.empty_cache()
    out["logits_path_other_vocabularies"] = {"peak_gbs": peak_gbs, "peak_kind": "of " + peak_kind, "by_V": vocab}

    # cfg 2: in place over the whole packed batch (the gradient overwrites the logits, so every timed
    # call sees the previous call's output as its logits: same bytes moved, values irrelevant to time)
    spec = synth.SPECS[2]
    batch = synth.make_batch(spec, dev)
    T, V = batch.T, spec.V
    mask, seq, n = rlf.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id)
    adv = rlf.rlf_group_advantage(batch.rewards, group_size=spec.group_size)
    ws = rlf.new_workspace(rlf.FN_LOGP_LOSS, T, V)
    logp = torch.empty(T, dtype=torch.float32, device=dev)
    loss = torch.empty(4, dtype=torch.float64, device=dev)
    ms = timed(lambda: rlf.rlf_grpo_logp_loss_fwd_bwd(batch.logits, batch.ids, seq, adv, batch.old_logp, batch.ref_logp,
                                                      mask, synth.EPS_CLIP, synth.BETA_KL, denom=n, in_place=True,
                                                      logp_out=logp, loss_out=loss, workspace=ws), steps)
    out["cfg2_ragged_in_place"] = {"T": T, "responses": batch.B, "ms": ms, "tokens_per_s": T / ms * 1e3,
                                   "logits_gbs": T * V * 4 / ms / 1e6, "logits_gb": T * V * 2 / 1e9}
    del batch, ws
    torch.cuda.empty_cache()

    # cfg 4, logits path: 8 micro-batches of one 8192-token response, global denominator
    spec = synth.SPECS[4]
    tok = synth.make_tokens(spec)
    T = len(tok.ids)
    ids = torch.from_numpy(tok.ids).to(dev)
    cu = torch.from_numpy(tok.cu_seqlens).to(dev)
    mask, seq, n = rlf.rlf_build_loss_mask(ids, cu, spec.open_id, spec.close_id)
    adv = rlf.rlf_group_advantage(torch.from_numpy(tok.rewards).to(dev), group_size=spec.group_size)
    mb = 8192
    logits = synth.make_logits(synth.scaled(spec, D=0), mb, dev)      # one micro-batch worth, reused
    grad = torch.empty_like(logits)
    old = torch.full((T,), -14.0, device=dev)
    ws = rlf.new_workspace(rlf.FN_LOGP_LOSS, mb, V)
    logp = torch.empty(mb, dtype=torch.float32, device=dev)

    def logits_path():
        for i in range(T // mb):
            sl = slice(i * mb, (i + 1) * mb)
            rlf.rlf_grpo_logp_loss_fwd_bwd(logits, ids[sl], seq[sl], adv, old[sl], old[sl], mask[sl], synth.EPS_CLIP,
                                           synth.BETA_KL, denom=n, grad_logits=grad, logp_out=logp, loss_out=loss,
                                           workspace=ws)
    ms = timed(logits_path, steps)
    out["cfg4_logits_path_8_microbatches"] = {"T": T, "ms": ms, "tokens_per_s": T / ms * 1e3,
                                              "logits_gbs": T * V * 4 / ms / 1e6}
    del logits, grad, ws
    torch.cuda.empty_cache()
    out["cfg4_fused_lmhead"] = time_fused_lmhead(rlf, dev, 2, 0, cfg=4)
    torch.cuda.empty_cache()

    # cfg 4, fused path as the recipe words it: 8 calls of one 8192-token response each, the batch's
    # token count as denominator, grad_W accumulated over the calls
    H, W = synth.make_hidden_and_head(spec, T, dev)
    ws = rlf.new_workspace(rlf.FN_FUSED_LMHEAD, mb, spec.V, spec.D, rlf.RLF_BF16, dev)
    gh = torch.empty((T, spec.D), dtype=torch.bfloat16, device=dev)
    gw = torch.empty((spec.V, spec.D), dtype=torch.float32, device=dev)
    logp_all = torch.empty(T, dtype=torch.float32, device=dev)
    old = torch.full((T,), -11.9, device=dev)

    def fused_micro():
        for i in range(T // mb):
            sl = slice(i * mb, (i + 1) * mb)
            rlf.rlf_fused_lmhead_grpo(H[sl], W, ids[sl], seq[sl], adv, old[sl], old[sl], mask[sl], synth.EPS_CLIP,
                                      synth.BETA_KL, denom=n, grad_hidden=gh[sl], grad_W=gw, accumulate_grad_W=i > 0,
                                      logp_out=logp_all[sl], loss_out=loss, workspace=ws)
    ms = timed(fused_micro, 2)
    live = int(mask.sum().item())
    out["cfg4_fused_lmhead_8_microbatches"] = {
        "T": T, "ms": ms, "tokens_per_s": T / ms * 1e3,
        "executed_tflops": 2.0 * spec.V * spec.D * (T + 2 * live) / ms / 1e9}
    print(json.dumps({"other_configs": out, "gpu_launches": rlf.launch_count()}))


def run_cuda(args):
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    if args.fused_phases:
        if dist_env()[0] == 0:
            run_fused_phases(args)
        return
    if args.fused_only or args.other_configs:
        if rank == 0:
            run_other_configs(args) if args.other_configs else run_fused_only(args)
        return
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2509_06980_b200 import binding as rlf

    spec = synth.scaled(synth.SPECS[1], seed=shard_seed(synth.SPECS[1].seed, rank))
    if args.tokens_per_response:
        spec = synth.scaled(spec, len_lo=args.tokens_per_response, len_hi=args.tokens_per_response)
    batch = synth.make_batch(spec, dev)
    T, V, B = batch.T, spec.V, batch.B
    G = batch.tokens.group_size

    # CPU baseline first (rank 0, one GPU only): the oracle on a bounded sample of this workload
    cpu_baseline = None
    if rank == 0 and world == 1 and args.cpu_seconds > 0:
        cpu_baseline = time_oracle(batch, args.cpu_seconds)

    grad = torch.empty_like(batch.logits)
    mask = torch.empty(T, dtype=torch.uint8, device=dev)
    seq_id = torch.empty(T, dtype=torch.int32, device=dev)
    n_tok = torch.empty(1, dtype=torch.int64, device=dev)
    adv = torch.empty(B, dtype=torch.float32, device=dev)
    logp = torch.empty(T, dtype=torch.float32, device=dev)
    loss = torch.empty(4, dtype=torch.float64, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = rlf.new_workspace(rlf.FN_LOGP_LOSS, T, V, 0, rlf.RLF_BF16, dev)

    def step(ev=None):
        rlf.rlf_build_loss_mask(batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id, mask_out=mask,
                                seq_id_out=seq_id, n_out=n_tok, dev_status=status)
        rlf.rlf_group_advantage(batch.rewards, group_size=G, eps=1e-6, adv_out=adv, dev_status=status)
        if ev is not None:
            ev[0].record()
        rlf.rlf_grpo_logp_loss_fwd_bwd(batch.logits, batch.ids, seq_id, adv, batch.old_logp, batch.ref_logp, mask,
                                       synth.EPS_CLIP, synth.BETA_KL, denom=n_tok, grad_logits=grad,
                                       logp_out=logp, loss_out=loss, workspace=ws, dev_status=status)
        if ev is not None:
            ev[1].record()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = rlf.launch_count()
    barrier()
    e0.record()
    for k in range(args.steps):
        step(kev[k])
    e1.record()
    barrier()
    launches = rlf.launch_count() - launches0
    ms_total = e0.elapsed_time(e1)
    kernel_ms = [a.elapsed_time(b) for a, b in kev]
    time.sleep(0.25)
    clocks = sampler.stop()
    if status.item() != 0:
        raise SystemExit("device status %d after the timed region" % status.item())

    ms_total_max = max_over_ranks(ms_total, world, dev)
    value = aggregate(T * args.steps, world, ms_total_max / 1e3)

    # the two launch-latency-bound calls of the step, each looped on its own (5 bytes per token; B floats)
    small_us = None
    if rank == 0 and world == 1:
        def loop_us(fn, reps=200):
            for _ in range(10):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) * 1e3 / reps
        small_us = {
            "rlf_build_loss_mask": loop_us(lambda: rlf.rlf_build_loss_mask(
                batch.ids, batch.cu_seqlens, spec.open_id, spec.close_id, mask_out=mask, seq_id_out=seq_id, n_out=n_tok,
                dev_status=status)),
            "rlf_group_advantage": loop_us(lambda: rlf.rlf_group_advantage(
                batch.rewards, group_size=G, eps=1e-6, adv_out=adv, dev_status=status)),
            "what": "microseconds per call, 200 calls back to back (launch-latency bound)"}

    # the same step looped back to back for about a second: the row kernel keeps the SMs busy enough to
    # reach the board's power cap, and what it holds then is lower than over 20 steps from a rested GPU
    sustained = None
    if rank == 0 and world == 1 and not args.tokens_per_response:
        n_sus = 300
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(n_sus // 2):
            step()
        s0.record()
        for _ in range(n_sus):
            step()
        s1.record()
        torch.cuda.synchronize()
        sus_ms = s0.elapsed_time(s1) / n_sus
        sustained = {"steps": n_sus, "after_untimed_steps": n_sus // 2, "ms_per_step": sus_ms,
                     "tokens_per_s": T / sus_ms * 1e3, "logits_gbs_whole_step": T * V * 4 / sus_ms / 1e6}

    # end to end through the host-buffer entry point: inputs start in pinned host memory, the loss
    # (and per-token log-probs) come back to the host, every step
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        h_logits = torch.empty((T, V), dtype=torch.bfloat16).pin_memory()
        h_logits.copy_(batch.logits)
        pin = lambda t: t.cpu().contiguous().pin_memory()
        h_ids, h_cu, h_rw = pin(batch.ids), pin(batch.cu_seqlens), pin(batch.rewards)
        h_old, h_ref = pin(batch.old_logp), pin(batch.ref_logp)
        h_loss = torch.zeros(4, dtype=torch.float64).pin_memory()
        h_logp = torch.zeros(T, dtype=torch.float32).pin_memory()
        h_st = torch.zeros(1, dtype=torch.int32).pin_memory()
        del grad
        arena = torch.empty(rlf.step_arena_bytes(T, V, B), dtype=torch.uint8, device=dev)

        def host_step():
            rlf.rlf_grpo_step_host(h_logits, h_ids, h_cu, G, h_rw, h_old, h_ref, spec.open_id, spec.close_id, 1e-6,
                                   synth.EPS_CLIP, synth.BETA_KL, h_loss, arena, h_logp_out=h_logp, h_dev_status=h_st)
        host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            host_step()              # waits for its stream before returning
        barrier()
        el = max_over_ranks(time.perf_counter() - t0, world, dev)
        h2d = T * V * 2 + T * 4 * 3 + (B + 1) * 4 + B * 4
        d2h = 4 * 8 + T * 4 + 4
        e2e = {"value": aggregate(T * e2e_steps, world, el), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "loss": float(h_loss[0].item())}

    # forward-only log-prob + entropy over the same logits (the old / reference policy pass): read-only
    fwd_only = None
    if rank == 0 and world == 1:
        ent = torch.empty(T, dtype=torch.float32, device=dev)
        ws_ent = rlf.new_workspace(rlf.FN_LOGP_ENTROPY, T, V, 0, rlf.RLF_BF16, dev)
        for _ in range(2):
            rlf.rlf_logp_entropy_fwd(batch.logits, batch.ids, logp_out=logp, entropy_out=ent, workspace=ws_ent)
        torch.cuda.synchronize()
        fe = []
        for _ in range(max(3, min(args.steps, 10))):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            rlf.rlf_logp_entropy_fwd(batch.logits, batch.ids, logp_out=logp, entropy_out=ent, workspace=ws_ent)
            b.record()
            torch.cuda.synchronize()
            fe.append(a.elapsed_time(b))
        fms = statistics.mean(fe)
        # log-prob alone (no entropy output): what the old / reference policy pass needs at the least
        for _ in range(2):
            rlf.rlf_logp_entropy_fwd(batch.logits, batch.ids, want_entropy=False, logp_out=logp, workspace=ws_ent)
        torch.cuda.synchronize()
        fl = []
        for _ in range(max(3, min(args.steps, 10))):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            rlf.rlf_logp_entropy_fwd(batch.logits, batch.ids, want_entropy=False, logp_out=logp, workspace=ws_ent)
            b.record()
            torch.cuda.synchronize()
            fl.append(a.elapsed_time(b))
        lms = statistics.mean(fl)
        hbm_peak, hbm_kind = _peaks()
        fwd_only = {"entry": "rlf_logp_entropy_fwd", "ms": fms, "tokens_per_s": T / fms * 1e3,
                    "logp_only": {"ms": lms, "gbs": T * V * 2 / lms / 1e6, "frac": T * V * 2 / lms / 1e6 / hbm_peak},
                    "roofline": {"bound": "hbm", "achieved": T * V * 2 / fms / 1e6, "peak": hbm_peak, "unit": "GB/s",
                                 "frac": T * V * 2 / fms / 1e6 / hbm_peak, "peak_kind": "of " + hbm_kind,
                                 "traffic": NCU_TRAFFIC_ENTROPY["dram_bytes_per_token"] * T
                                 if NCU_TRAFFIC_ENTROPY["section_sha1"] == _entropy_section_sha1() else None,
                                 "algorithmic_bytes": T * V * 2}}

    # skip-masked variant on the same batch: rows without loss weight are neither read nor computed
    skip_masked = None
    if rank == 0 and world == 1:
        g2 = torch.empty_like(batch.logits)
        skip_masked = {"entry": "rlf_grpo_logp_loss_fwd_bwd_skip_masked", "live_fraction": float(mask.float().mean().item())}
        for zero in (True, False):
            def run_skip():
                rlf.rlf_grpo_logp_loss_fwd_bwd_skip_masked(batch.logits, batch.ids, seq_id, adv, batch.old_logp,
                                                           batch.ref_logp, mask, synth.EPS_CLIP, synth.BETA_KL,
                                                           denom=n_tok, grad_logits=g2, zero_masked_grad=zero,
                                                           logp_out=logp, loss_out=loss, workspace=ws)
            for _ in range(2):
                run_skip()
            torch.cuda.synchronize()
            ts = []
            for _ in range(max(3, min(args.steps, 10))):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                run_skip()
                b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            sms = statistics.mean(ts)
            n_live = int(mask.sum().item())
            moved = n_live * V * 4 + ((T - n_live) * V * 2 if zero else 0)
            skip_masked["zero_fill" if zero else "no_fill"] = {"ms": sms, "tokens_per_s": T / sms * 1e3,
                                                               "algorithmic_bytes": moved, "gbs": moved / sms / 1e6}
        del g2

    # context for the roofline fraction: the same STREAM-style copy that produced the recorded peak,
    # taken on this GPU in this run (GPUs of one pool differ by a few per cent)
    copy_gbs = None
    if rank == 0 and world == 1 and not args.tokens_per_response:
        src = torch.empty(1 << 30, dtype=torch.bfloat16, device=dev)
        dst = torch.empty_like(src)
        src.zero_()
        best = None
        for i in range(12):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            dst.copy_(src)
            b.record()
            torch.cuda.synchronize()
            if i >= 2:
                best = a.elapsed_time(b) if best is None else min(best, a.elapsed_time(b))
        copy_gbs = 2 * src.numel() * 2 / best / 1e6
        del src, dst
        torch.cuda.empty_cache()

    fused = None
    if rank == 0 and world == 1 and not args.skip_fused:
        fused = time_fused_lmhead(rlf, dev, max(2, min(args.steps, 5)))

    if rank != 0:
        return
    peak, peak_kind = _peaks()
    k_ms = statistics.mean(kernel_ms)
    alg_bytes = T * V * 4                      # bf16 logits read once + bf16 grad written once
    achieved = alg_bytes / (k_ms * 1e-3) / 1e9
    traffic = None
    if NCU_TRAFFIC["dram_bytes_per_token"] and NCU_TRAFFIC["logits_loss_cu_sha1"] == _kernel_sha1():
        traffic = NCU_TRAFFIC["dram_bytes_per_token"] * T
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_total_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": workload_config(world, args.tokens_per_response),
        "arithmetic": "bf16 in/out, fp32 accumulate, fp64 loss sum",
        "l2": "inputs (%.1f GB per step) exceed L2; no flush needed" % (T * V * 2 / 1e9),
        "grad": "out of place",
        "logits_gbs": achieved,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": "of " + peak_kind, "frac_of_nominal_8tbs": achieved / 8000.0, "traffic": traffic,
                     "kernel": "grpo_row_cluster_kernel (timed as the rlf_grpo_logp_loss_fwd_bwd call: "
                               "row kernel + 3 sub-10us kernels)",
                     "kernel_ms": k_ms, "kernel_ms_min": min(kernel_ms), "algorithmic_bytes": alg_bytes,
                     "copy_gbs_this_gpu": copy_gbs,
                     "frac_of_copy_this_gpu": (achieved / copy_gbs) if copy_gbs else None},
        "gpu_launches": int(launches),
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                   "samples": clocks["samples"]},
        "loss": float(loss[0].item()),
        "sustained": sustained,
        "small_calls_us": small_us,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline
    if fwd_only is not None:
        line["logp_entropy_fwd"] = fwd_only
    if skip_masked is not None:
        line["skip_masked"] = skip_masked
    if fused is not None:
        line["fused_lmhead"] = fused
    print(json.dumps(line))


def launch_ranks(n):
    """Re-run this command line as n ranks (one per GPU) under torch.distributed.run on this node and
    return its exit code; rank 0 of that job prints the JSON line."""
    import socket
    import subprocess
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="time budget of the CPU-oracle baseline leg")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--skip-fused", action="store_true", help="do not time the fused LM-head variant")
    ap.add_argument("--fused-only", action="store_true", help="time only the fused LM-head variant (rank 0)")
    ap.add_argument("--other-configs", action="store_true",
                    help="time cfg 2 (ragged, in place) and cfg 4 (micro-batched; both paths) instead (rank 0)")
    ap.add_argument("--tokens-per-response", type=int, default=0,
                    help="smaller micro-batch of the same recipe (profiling captures); 0 = the full 2048")
    ap.add_argument("--fused-phases", action="store_true",
                    help="sustained cost of the fused LM-head call by phase, with clocks and power (rank 0)")
    ap.add_argument("--phase-seconds", type=float, default=3.0)
    ap.add_argument("--fused-cfg", type=int, default=3, choices=[3, 4],
                    help="with --fused-only: the Qwen3-4B head (3) or the Qwen3-8B head (4)")
    ap.add_argument("--responses", type=int, default=0,
                    help="with --fused-only: one group of this many full-length responses (profiling captures)")
    ap.add_argument("--source-keys", action="store_true",
                    help="print the source hashes that key the stored ncu traffic figures, and exit")
    args = ap.parse_args()
    if args.source_keys:
        print(json.dumps({"logits_loss_cu_sha1 (row kernel section)": _kernel_sha1(),
                          "section_sha1 (forward-only section)": _entropy_section_sha1(),
                          "lmhead_cu_sha1": _lmhead_sha1()}))
        return
    if args.gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    world_env = os.environ.get("WORLD_SIZE")
    if args.impl == "cuda" and world_env is None and args.gpus > 1:
        # started as a plain process: become the launcher of one rank per GPU
        raise SystemExit(launch_ranks(args.gpus))
    if args.impl == "cuda" and int(world_env or "1") != args.gpus:
        raise SystemExit("bench.py: --gpus %d but WORLD_SIZE=%s; refusing to report a line whose n_gpus is not "
                         "the number of ranks that ran" % (args.gpus, world_env))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)
        if int(os.environ.get("WORLD_SIZE", "1")) > 1:
            import torch.distributed as dist
            if dist.is_initialized():
                dist.destroy_process_group()


if __name__ == "__main__":
    main()
