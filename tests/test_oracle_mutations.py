"""Sharpness of the oracle's pins: plant one plausible mistake at a time in a copy of the oracle's
source (on the CPU, never in the CUDA path), build it, and check that the pin tests of the affected
function fail.  A mutation that every pin lets through would mean the oracle is not pinned there."""
import os
import subprocess
import sys
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "rlf_oracle.c")

# (name, text to replace, replacement, pin file that must catch it)
MUTATIONS = [
    ("close_marker_not_masked", "inside = 0;\n                m = 0;", "inside = 0;\n                m = 1;", "test_oracle_mask.py"),
    ("state_leaks_across_sequences", "        int inside = 0;\n        for (int64_t t = cu_seqlens[b]", "        static int inside = 0;\n        for (int64_t t = cu_seqlens[b]", "test_oracle_mask.py"),
    ("stray_close_opens_nothing_but_is_masked", "m = inside ? 0 : 1;", "m = (inside || ids[t] == close_id) ? 0 : 1;", "test_oracle_mask.py"),
    ("biased_std_always", "double div = unbiased ? (double)(n - 1) : (double)n;", "double div = (double)n;", "test_oracle_advantage.py"),
    ("advantage_not_centred", "? ((double)rewards[i] - mean) / (sd + eps) : 0.0;", "? ((double)rewards[i]) / (sd + eps) : 0.0;", "test_oracle_advantage.py"),
    ("degenerate_group_divides_zero_by_zero", "adv[i] = (sd + eps > 0.0) ? ((double)rewards[i] - mean) / (sd + eps) : 0.0;", "adv[i] = ((double)rewards[i] - mean) / (sd + eps);", "test_oracle_advantage.py"),
    ("clip_uses_wrong_side", "*clipped = (A > 0.0 && rho > hi) || (A < 0.0 && rho < lo);", "*clipped = (A > 0.0 && rho < lo) || (A < 0.0 && rho > hi);", "test_oracle_loss.py"),
    ("kl_gradient_sign", "*dkl = 1.0 - exp(d);", "*dkl = exp(d) - 1.0;", "test_oracle_loss.py"),
    ("kl_direction", "double d = ref_lp - logp;", "double d = logp - ref_lp;", "test_oracle_loss.py"),
    ("beta_dropped_from_gradient", "double g = w * (dpg + beta_kl * dkl);", "double g = w * (dpg);", "test_oracle_loss.py"),
    ("max_not_subtracted_in_sum", "s += exp(widen(logits, dtype, off + v) - m);", "s += exp(widen(logits, dtype, off + v));", "test_oracle_loss.py"),
    ("onehot_sign", "grad[t * (int64_t)V + v] = g * ((v == y ? 1.0 : 0.0) - p);", "grad[t * (int64_t)V + v] = g * ((v == y ? 1.0 : 0.0) + p);", "test_oracle_loss.py"),
    ("denominator_ignores_override", "if (denom >= 0) n = denom;", "", "test_oracle_loss.py"),
    ("head_transposed", "widen(W, ORC_BF16, v * (int64_t)D + k);\n            z[t", "widen(W, ORC_BF16, (v * (int64_t)D + k) % ((int64_t)V * D - 1));\n            z[t", "test_oracle_fused.py"),
    ("grad_W_uses_wrong_operand", "acc += gz[t * (int64_t)V + v] * widen(hidden, ORC_BF16, t * (int64_t)D + k);", "acc += gz[t * (int64_t)V + v] * widen(hidden, ORC_BF16, t * (int64_t)D + (D - 1 - k));", "test_oracle_fused.py"),
    ("asymmetric_clip_uses_low_for_both", "1.0 - eps_low, 1.0 + eps_high, &pg", "1.0 - eps_low, 1.0 + eps_low, &pg", "test_oracle_objective.py"),
    ("sequence_mean_weighs_by_batch_count", "w[t] = mask[t] ? 1.0 / ((double)nb[seq_id[t]] * sd) : 0.0;", "w[t] = mask[t] ? 1.0 / ((double)T * sd) : 0.0;", "test_oracle_objective.py"),
    ("kl_reward_counts_masked_tokens", "            if (!mask[t])\n                continue;\n            double d = (double)old_logp[t]", "            double d = (double)old_logp[t]", "test_oracle_kl_reward.py"),
    ("kl_reward_k3_direction", "k = exp(-d) + d - 1.0;", "k = exp(d) - d - 1.0;", "test_oracle_kl_reward.py"),
    ("kl_reward_penalty_sign", "reward_out[b] = (double)rewards[b] - beta * acc;", "reward_out[b] = (double)rewards[b] + beta * acc;", "test_oracle_kl_reward.py"),
    ("entropy_sign", "if (pv > 0.0) h -= pv * lp;", "if (pv > 0.0) h += pv * lp;", "test_oracle_entropy.py"),
]


@pytest.mark.parametrize("name,old,new,pin_file", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(name, old, new, pin_file):
    src = open(SRC).read()
    assert src.count(old) >= 1, "mutation target not found: " + name
    mutated = src.replace(old, new, 1)
    with tempfile.TemporaryDirectory() as td:
        c = os.path.join(td, "mutant.c")
        so = os.path.join(td, "mutant.so")
        open(c, "w").write(mutated)
        subprocess.check_call(["gcc", "-O1", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", so, c, "-lm"])
        env = dict(os.environ, RLF_ORACLE_LIB=so)
        r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", pin_file), "-x", "-q",
                            "-p", "no:cacheprovider"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert r.returncode != 0, "no pin noticed the planted mistake '%s'" % name
    assert "failed" in r.stdout or "error" in r.stdout.lower()
