"""B200-native GRPO policy-update loss path: observation-marker loss mask,
group-relative advantages, fused log-prob + clipped-ratio + k3-KL loss with
grad_logits, and the fused LM-head variant, behind a C-ABI CUDA library.

`synth` (input generators) imports without the CUDA library; `binding` loads
the library and fails loudly when it is missing."""
__all__ = ["synth", "binding"]
