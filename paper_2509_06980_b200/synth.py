"""Seeded synthetic inputs shaped like multi-turn tool-use GRPO batches.

This module only *draws inputs*: packed response token streams with
tool-observation spans between marker ids, per-response rewards, logits or
hidden states / LM-head weights, and behaviour / reference log-probs placed
near the current policy's.  It contains none of the loss path's arithmetic and
is the one module that both the CPU oracle's tests and the CUDA path's tests
and benchmark draw from, so that both sides see identical bytes.

The only library maths used is ``torch.log_softmax`` in ``center_logp``: the
recipe asks for ``old_logp = new_logp + noise`` and ``ref_logp = new_logp +
noise``, so the generator needs *a* value of new_logp to centre the noise on.
It is an input-synthesis step: whatever it returns is handed, as data, to both
implementations.

Recipes (second argument of N(.,.) is a standard deviation):
  cfg 0  16 responses (4 prompts x G=4) of 64 tokens, 2 observation spans each of
         4..12 tokens (+2 markers), V=1024, fp32 logits ~ N(0,2), Bernoulli(0.5) rewards.
  cfg 1  16 responses (2 x G=8) of 2048 tokens, 3..4 spans of 100..400 tokens,
         V=151936, bf16 logits ~ N(0,3), U[0,1] rewards.
  cfg 2  64 responses (8 x G=8), lengths U{256..4096} packed with int32 cu_seqlens,
         1..6 spans covering a fraction U(0.2,0.6) of each response, V=151936 bf16.
  cfg 3  as cfg 1 (same tokens, masks, rewards) with hidden [T,2560] ~ N(0,1) and
         W [151936,2560] ~ N(0,0.02) in place of logits.
  cfg 4  8 responses (1 x G=8) of 8192 tokens, 6..10 spans of 100..600 tokens,
         hidden [T,4096], W [151936,4096]; processed as 8 micro-batches of one response.
Marker ids are 1000 (open) / 1001 (close) (the last two ids of the vocabulary in
reduced-size test recipes whose vocabulary is smaller); filler ids are uniform
over the vocabulary minus the two markers.  eps_clip = 0.2, beta_kl = 0.001,
old = new + N(0,0.05), ref = new + N(0,0.1) throughout.
"""
from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

OPEN_ID = 1000
CLOSE_ID = 1001
EPS_CLIP = 0.2
BETA_KL = 0.001
V_QWEN3 = 151936


@dataclass
class Spec:
    name: str
    seed: int
    num_prompts: int
    group_size: int
    len_lo: int
    len_hi: int            # response length ~ U{len_lo..len_hi}
    spans_lo: int
    spans_hi: int          # spans per response ~ U{spans_lo..spans_hi}
    obs_lo: int = 0
    obs_hi: int = 0        # observation tokens per span ~ U{obs_lo..obs_hi} (markers extra)
    cover_lo: float = 0.0
    cover_hi: float = 0.0  # if > 0: spans cover this fraction of the response instead
    V: int = V_QWEN3
    logits_dtype: str = "bf16"
    logits_std: float = 3.0
    reward: str = "uniform"   # or "bernoulli"
    D: int = 0               # hidden size for the fused LM-head variant (0 = logits given)
    w_std: float = 0.02

    @property
    def open_id(self):
        """1000 where the vocabulary has it; the second-to-last id in smaller test vocabularies."""
        return OPEN_ID if self.V > CLOSE_ID else max(self.V - 2, 0)

    @property
    def close_id(self):
        return CLOSE_ID if self.V > CLOSE_ID else max(self.V - 1, 0)

    @property
    def has_spans(self):
        return self.V >= 4


SPECS = {
    0: Spec("cfg0_tiny", 0, 4, 4, 64, 64, 2, 2, obs_lo=4, obs_hi=12, V=1024,
            logits_dtype="f32", logits_std=2.0, reward="bernoulli"),
    1: Spec("cfg1_qwen3_4b_microbatch", 1, 2, 8, 2048, 2048, 3, 4, obs_lo=100, obs_hi=400),
    2: Spec("cfg2_ragged_varlen", 2, 8, 8, 256, 4096, 1, 6, cover_lo=0.2, cover_hi=0.6),
    3: Spec("cfg3_fused_lmhead_4b", 1, 2, 8, 2048, 2048, 3, 4, obs_lo=100, obs_hi=400, D=2560),
    4: Spec("cfg4_qwen3_8b_longctx", 4, 1, 8, 8192, 8192, 6, 10, obs_lo=100, obs_hi=600, D=4096),
}


def scaled(spec: Spec, **kw) -> Spec:
    """A copy of a recipe with some sizes overridden (reduced-size parity cases)."""
    d = dict(spec.__dict__)
    d.update(kw)
    return Spec(**d)


def _composition(rng, total, parts, minimum):
    """`parts` integers >= minimum that sum to `total`, uniformly at random."""
    free = total - parts * minimum
    assert free >= 0
    if parts == 1:
        return np.array([total], dtype=np.int64)
    cuts = np.sort(rng.integers(0, free + 1, size=parts - 1))
    sizes = np.diff(np.concatenate([[0], cuts, [free]])) + minimum
    return sizes.astype(np.int64)


def place_spans(rng, length, obs_lens):
    """Start offsets of non-overlapping spans (each obs_len + 2 marker tokens) inside a
    response of `length` tokens, with at least one model token before, between and after."""
    k = len(obs_lens)
    used = int(sum(obs_lens)) + 2 * k
    gaps = _composition(rng, length - used, k + 1, 1)
    starts, pos = [], 0
    for j in range(k):
        pos += int(gaps[j])
        starts.append(pos)
        pos += int(obs_lens[j]) + 2
    return starts


@dataclass
class Tokens:
    ids: np.ndarray            # int32 [T] target token ids, markers placed
    cu_seqlens: np.ndarray     # int32 [B+1]
    rewards: np.ndarray        # float32 [B]
    group_size: int
    n_span_tokens: int         # observation tokens + markers, all responses
    spans: list = field(default_factory=list)   # (response, start, obs_len)


def make_tokens(spec: Spec) -> Tokens:
    rng = np.random.default_rng(1000 + spec.seed)
    B = spec.num_prompts * spec.group_size
    lens = rng.integers(spec.len_lo, spec.len_hi + 1, size=B)
    cu = np.zeros(B + 1, dtype=np.int64)
    cu[1:] = np.cumsum(lens)
    T = int(cu[-1])
    open_id, close_id = spec.open_id, spec.close_id
    if spec.has_spans:
        # draw from the vocabulary minus the two marker ids, so that spans are exactly the ones placed
        ids = rng.integers(0, spec.V - 2, size=T).astype(np.int64)
        ids = np.where(ids >= open_id, ids + 1, ids)
        ids = np.where(ids >= close_id, ids + 1, ids)
    else:
        ids = rng.integers(0, spec.V, size=T).astype(np.int64)
    assert ids.min(initial=0) >= 0 and ids.max(initial=0) < spec.V
    spans, n_span = [], 0
    for b in range(B):
        L = int(lens[b])
        k = int(rng.integers(spec.spans_lo, spec.spans_hi + 1)) if spec.has_spans else 0
        if spec.cover_hi > 0:
            frac = rng.uniform(spec.cover_lo, spec.cover_hi)
            covered = max(int(round(frac * L)), 3 * k)
            covered = min(covered, L - (k + 1))
            per_span = _composition(rng, covered, k, 3)   # each >= 1 obs token + 2 markers
            obs = [int(x) - 2 for x in per_span]
        else:
            obs = [int(x) for x in rng.integers(spec.obs_lo, spec.obs_hi + 1, size=k)]
            while sum(obs) + 2 * k + (k + 1) > L:        # reduced-size cases: shrink to fit
                if all(x == 1 for x in obs):             # even one-token spans do not fit: one span fewer
                    obs, k = obs[:-1], k - 1
                else:
                    obs = [max(1, x // 2) for x in obs]
        starts = place_spans(rng, L, obs)
        for s, n in zip(starts, obs):
            a = int(cu[b]) + s
            ids[a] = open_id
            ids[a + n + 1] = close_id
            spans.append((b, s, n))
            n_span += n + 2
    if spec.reward == "bernoulli":
        rewards = (rng.random(B) < 0.5).astype(np.float32)
    else:
        rewards = rng.random(B).astype(np.float32)
    return Tokens(ids.astype(np.int32), cu.astype(np.int32), rewards, spec.group_size, n_span, spans)


def _torch_gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_logits(spec: Spec, T: int, device="cpu", row_chunk=2048) -> torch.Tensor:
    """[T, V] logits ~ N(0, logits_std) in the recipe's dtype, drawn chunk by chunk."""
    dt = torch.bfloat16 if spec.logits_dtype == "bf16" else torch.float32
    g = _torch_gen(2000 + spec.seed, device)
    out = torch.empty((T, spec.V), dtype=dt, device=device)
    for r0 in range(0, T, row_chunk):
        r1 = min(T, r0 + row_chunk)
        blk = torch.randn((r1 - r0, spec.V), generator=g, device=device, dtype=torch.float32)
        out[r0:r1] = (blk * spec.logits_std).to(dt)
    return out


def make_hidden_and_head(spec: Spec, T: int, device="cpu"):
    """hidden [T, D] ~ N(0,1) and LM-head weight W [V, D] ~ N(0, w_std), both bf16."""
    g = _torch_gen(3000 + spec.seed, device)
    hidden = torch.randn((T, spec.D), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    W = torch.empty((spec.V, spec.D), dtype=torch.bfloat16, device=device)
    step = 16384
    for v0 in range(0, spec.V, step):
        v1 = min(spec.V, v0 + step)
        W[v0:v1] = (torch.randn((v1 - v0, spec.D), generator=g, device=device,
                                dtype=torch.float32) * spec.w_std).to(torch.bfloat16)
    return hidden, W


def center_logp(logits: torch.Tensor, ids: torch.Tensor, row_chunk=1024) -> torch.Tensor:
    """A library value of the current policy's log-prob of each target token, used only
    as the centre of the noise that makes old_logp / ref_logp (input synthesis)."""
    T = logits.shape[0]
    out = torch.empty(T, dtype=torch.float32, device=logits.device)
    idx = ids.to(device=logits.device, dtype=torch.int64).clamp(0, logits.shape[1] - 1)
    for r0 in range(0, T, row_chunk):
        r1 = min(T, r0 + row_chunk)
        lp = torch.log_softmax(logits[r0:r1].float(), dim=-1)
        out[r0:r1] = lp.gather(1, idx[r0:r1, None])[:, 0]
    return out


def center_logp_from_head(hidden, W, ids, row_chunk=512) -> torch.Tensor:
    """Same as center_logp with the logits formed by a library matmul (bf16 in, fp32 out)."""
    T = hidden.shape[0]
    out = torch.empty(T, dtype=torch.float32, device=hidden.device)
    idx = ids.to(device=hidden.device, dtype=torch.int64).clamp(0, W.shape[0] - 1)
    Wf = W.float() if hidden.device.type == "cpu" else None
    for r0 in range(0, T, row_chunk):
        r1 = min(T, r0 + row_chunk)
        if Wf is not None:
            z = hidden[r0:r1].float() @ Wf.t()
        else:
            z = (hidden[r0:r1] @ W.t()).float()
        lp = torch.log_softmax(z, dim=-1)
        out[r0:r1] = lp.gather(1, idx[r0:r1, None])[:, 0]
    return out


def perturbed_logps(spec: Spec, center: torch.Tensor):
    """old_logp = center + N(0,0.05), ref_logp = center + N(0,0.1), fp32, on center's device."""
    rng = np.random.default_rng(4000 + spec.seed)
    T = center.shape[0]
    n_old = torch.from_numpy(rng.normal(0.0, 0.05, size=T).astype(np.float32)).to(center.device)
    n_ref = torch.from_numpy(rng.normal(0.0, 0.10, size=T).astype(np.float32)).to(center.device)
    return (center + n_old).contiguous(), (center + n_ref).contiguous()


@dataclass
class Batch:
    spec: Spec
    tokens: Tokens
    ids: torch.Tensor                  # int32 [T]
    cu_seqlens: torch.Tensor           # int32 [B+1]
    rewards: torch.Tensor              # fp32 [B]
    old_logp: torch.Tensor             # fp32 [T]
    ref_logp: torch.Tensor             # fp32 [T]
    logits: Optional[torch.Tensor] = None    # [T, V]
    hidden: Optional[torch.Tensor] = None    # bf16 [T, D]
    W: Optional[torch.Tensor] = None         # bf16 [V, D]

    @property
    def T(self):
        return int(self.ids.shape[0])

    @property
    def B(self):
        return int(self.rewards.shape[0])


def make_batch(spec: Spec, device="cpu", with_logits=True) -> Batch:
    """Draw every input of one policy-update step for a recipe, on `device`."""
    tok = make_tokens(spec)
    T = int(tok.ids.shape[0])
    ids = torch.from_numpy(tok.ids).to(device)
    cu = torch.from_numpy(tok.cu_seqlens).to(device)
    rewards = torch.from_numpy(tok.rewards).to(device)
    logits = hidden = W = None
    if spec.D > 0:
        hidden, W = make_hidden_and_head(spec, T, device)
        center = center_logp_from_head(hidden, W, ids)
        if with_logits:
            logits = None
    else:
        logits = make_logits(spec, T, device)
        center = center_logp(logits, ids)
    old_lp, ref_lp = perturbed_logps(spec, center)
    return Batch(spec, tok, ids, cu, rewards, old_lp, ref_lp, logits, hidden, W)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 array of its bit patterns (CPU copy)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def as_oracle_array(t: torch.Tensor) -> np.ndarray:
    """Tensor -> numpy array holding the same bytes (bf16 as uint16 bit patterns)."""
    if t.dtype == torch.bfloat16:
        return bf16_bits(t)
    return t.detach().cpu().contiguous().numpy()
