"""Thin ctypes binding of the C-ABI CUDA library (include/rlf.h).

Argument marshalling only: every function takes torch tensors (device memory and
streams are PyTorch's), checks dtypes / devices, and passes raw pointers to the
entry point of the same name.  Nothing is computed here and there is no fallback:
importing this module raises if the library has not been built.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "librlf.so")

RLF_BF16, RLF_F32 = 0, 1
FN_LOGP_LOSS, FN_FUSED_LMHEAD, FN_LOGP_ENTROPY, FN_FUSED_LOGP_ENTROPY = 3, 4, 5, 6
DEV_BAD_TARGET, DEV_BAD_SEQ, DEV_NONFINITE, DEV_TIMEOUT = 1, 2, 4, 8

EXPORTS = [
    "rlf_build_loss_mask", "rlf_count_live_responses", "rlf_group_advantage", "rlf_rule_reward", "rlf_kl_in_reward", "rlf_grpo_logp_loss_fwd_bwd",
    "rlf_grpo_logp_loss_fwd_bwd_static", "rlf_grpo_logp_loss_fwd_bwd_skip_masked", "rlf_grpo_logp_loss_fwd_bwd_obj", "rlf_logp_entropy_fwd", "rlf_fused_lmhead_grpo", "rlf_fused_lmhead_grpo_obj", "rlf_fused_lmhead_logp_entropy", "rlf_workspace_bytes", "rlf_grpo_step_host", "rlf_step_arena_bytes",
    "rlf_tune_logits_kernel", "rlf_tune_logits_grid", "rlf_tune_lmhead", "rlf_tune_lmhead_schedule", "rlf_tune_lmhead_backward", "rlf_tune_lmhead_pacing", "rlf_launch_count", "rlf_status_string", "rlf_version",
]

if not os.path.exists(_LIB_PATH):
    raise ImportError(
        "CUDA library %s is missing: build it with `python -m paper_2509_06980_b200.build` "
        "(there is no CPU fallback)" % _LIB_PATH)

_lib = ctypes.CDLL(_LIB_PATH)

_vp, _i32, _i64, _f32, _sz, _int = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float,
                                    ctypes.c_size_t, ctypes.c_int)
_lib.rlf_build_loss_mask.argtypes = [_vp, _vp, _i32, _i64, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.rlf_count_live_responses.argtypes = [_vp, _vp, _i32, _i64, _vp, _vp, _vp]
_lib.rlf_group_advantage.argtypes = [_vp, _vp, _i32, _i32, _f32, _int, _vp, _vp, _vp]
_lib.rlf_grpo_logp_loss_fwd_bwd.argtypes = [_vp, _int, _i64, _i32, _i64, _vp, _vp, _vp, _i32, _vp, _vp, _vp,
                                            _f32, _f32, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.rlf_grpo_logp_loss_fwd_bwd_static.argtypes = [_vp, _int, _i64, _i32, _i64, _vp, _vp, _vp, _i32, _vp, _vp, _vp,
                                                   _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.rlf_grpo_logp_loss_fwd_bwd_static.restype = _int
_lib.rlf_fused_lmhead_grpo.argtypes = [_vp, _vp, _i64, _i32, _i32, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _f32,
                                       _f32, _vp, _vp, _vp, _vp, _vp, _int, _vp, _sz, _vp, _vp]
_lib.rlf_workspace_bytes.argtypes = [_int, _i64, _i32, _i32, _int]
_lib.rlf_workspace_bytes.restype = _sz
_lib.rlf_grpo_step_host.argtypes = [_vp, _int, _i64, _i32, _vp, _vp, _i32, _i32, _vp, _vp, _vp, _i32, _i32,
                                    _f32, _f32, _f32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.rlf_step_arena_bytes.argtypes = [_i64, _i32, _i32, _int]
_lib.rlf_step_arena_bytes.restype = _sz
_lib.rlf_tune_logits_kernel.argtypes = [_int, _int, _int]
_lib.rlf_launch_count.restype = _i64
_lib.rlf_status_string.argtypes = [_int]
_lib.rlf_status_string.restype = ctypes.c_char_p
_lib.rlf_version.restype = _int
_lib.rlf_tune_logits_grid.argtypes = [_int, _int]
_lib.rlf_tune_lmhead.argtypes = [_int]
_lib.rlf_tune_lmhead_schedule.argtypes = [_int, _int, _int]
_lib.rlf_tune_lmhead_backward.argtypes = [_int, _int]
_lib.rlf_tune_lmhead_pacing.argtypes = [_int]
_lib.rlf_rule_reward.argtypes = [_vp, _vp, _i32, _i32, _vp, _vp]
_lib.rlf_kl_in_reward.argtypes = [_vp, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _int, _vp, _vp, _vp, _vp]
_lib.rlf_grpo_logp_loss_fwd_bwd_obj.argtypes = [_vp, _int, _i64, _i32, _i64, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _f32,
                                                _f32, _f32, _int, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.rlf_grpo_logp_loss_fwd_bwd_skip_masked.argtypes = [_vp, _int, _i64, _i32, _i64, _vp, _vp, _vp, _i32, _vp, _vp, _vp,
                                                        _f32, _f32, _vp, _vp, _vp, _vp, _int, _vp, _sz, _vp, _vp]
_lib.rlf_logp_entropy_fwd.argtypes = [_vp, _int, _i64, _i32, _i64, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.rlf_fused_lmhead_grpo_obj.argtypes = [_vp, _vp, _i64, _i32, _i32, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _f32, _f32,
                                           _f32, _int, _int, _vp, _vp, _vp, _vp, _vp, _int, _vp, _sz, _vp, _vp]
_lib.rlf_fused_lmhead_logp_entropy.argtypes = [_vp, _vp, _i64, _i32, _i32, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
# every entry point that returns an rlf_status
for _n in ("rlf_build_loss_mask", "rlf_count_live_responses", "rlf_group_advantage", "rlf_rule_reward", "rlf_kl_in_reward",
           "rlf_grpo_logp_loss_fwd_bwd", "rlf_grpo_logp_loss_fwd_bwd_obj", "rlf_grpo_logp_loss_fwd_bwd_skip_masked",
           "rlf_logp_entropy_fwd", "rlf_fused_lmhead_grpo", "rlf_fused_lmhead_grpo_obj",
           "rlf_fused_lmhead_logp_entropy", "rlf_grpo_step_host", "rlf_tune_logits_kernel", "rlf_tune_logits_grid",
           "rlf_tune_lmhead", "rlf_tune_lmhead_schedule", "rlf_tune_lmhead_backward", "rlf_tune_lmhead_pacing"):
    getattr(_lib, _n).restype = _int


class RlfError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, _lib.rlf_status_string(code).decode(), code))


def _check(code, where):
    if code != 0:
        raise RlfError(code, where)


def _ptr(t, dtype=None, cuda=True):
    if t is None:
        return None
    if dtype is not None and t.dtype != dtype:
        raise TypeError("expected %s, got %s" % (dtype, t.dtype))
    if cuda and not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not cuda and t.is_cuda:
        raise ValueError("expected a host tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _dt(t):
    if t.dtype == torch.bfloat16:
        return RLF_BF16
    if t.dtype == torch.float32:
        return RLF_F32
    raise TypeError("logits must be bfloat16 or float32")


def version():
    return int(_lib.rlf_version())


def launch_count():
    return int(_lib.rlf_launch_count())


def status_string(code):
    return _lib.rlf_status_string(int(code)).decode()


def workspace_bytes(which_fn, T, V, D=0, dt=RLF_BF16):
    return int(_lib.rlf_workspace_bytes(which_fn, T, V, D, dt))


def new_workspace(which_fn, T, V, D=0, dt=RLF_BF16, device="cuda"):
    n = max(workspace_bytes(which_fn, T, V, D, dt), 256)
    return torch.empty(n, dtype=torch.uint8, device=device)


def tune_logits_kernel(cluster_ctas=0, threads_per_cta=0, one_exp=-1):
    _check(_lib.rlf_tune_logits_kernel(cluster_ctas, threads_per_cta, one_exp), "rlf_tune_logits_kernel")


def tune_logits_grid(rows_per_cluster=0, units_per_cta=0):
    _check(_lib.rlf_tune_logits_grid(int(rows_per_cluster), int(units_per_cta)), "rlf_tune_logits_grid")


def tune_lmhead(pair_ctas=1):
    _check(_lib.rlf_tune_lmhead(int(pair_ctas)), "rlf_tune_lmhead")


def tune_lmhead_backward(row_reference=1, two_accumulators=1):
    _check(_lib.rlf_tune_lmhead_backward(int(row_reference), int(two_accumulators)), "rlf_tune_lmhead_backward")


def tune_lmhead_pacing(on=1):
    _check(_lib.rlf_tune_lmhead_pacing(int(on)), "rlf_tune_lmhead_pacing")


def tune_lmhead_schedule(m_block=0, max_workers=0, chunk_tiles=0):
    _check(_lib.rlf_tune_lmhead_schedule(int(m_block), int(max_workers), int(chunk_tiles)),
           "rlf_tune_lmhead_schedule")


def rlf_build_loss_mask(ids, cu_seqlens, open_id, close_id, valid=None, mask_out=None, seq_id_out=None,
                        n_out=None, dev_status=None, want_seq_id=True):
    """-> (mask u8[T], seq_id i32[T] | None, n i64[1]) on the device."""
    T = ids.shape[0]
    B = cu_seqlens.shape[0] - 1
    dev = ids.device
    if mask_out is None:
        mask_out = torch.empty(T, dtype=torch.uint8, device=dev)
    if seq_id_out is None and want_seq_id:
        seq_id_out = torch.empty(T, dtype=torch.int32, device=dev)
    if n_out is None:
        n_out = torch.empty(1, dtype=torch.int64, device=dev)
    _check(_lib.rlf_build_loss_mask(_ptr(ids, torch.int32), _ptr(cu_seqlens, torch.int32), B, T, open_id,
                                    close_id, _ptr(valid, torch.uint8), _ptr(mask_out, torch.uint8),
                                    _ptr(seq_id_out, torch.int32), _ptr(n_out, torch.int64),
                                    _ptr(dev_status, torch.int32), _stream()), "rlf_build_loss_mask")
    return mask_out, seq_id_out, n_out


def rlf_count_live_responses(mask, cu_seqlens, count_out=None, dev_status=None):
    """-> int64[1] on the device: responses with at least one token of mask 1."""
    T = mask.shape[0]
    B = cu_seqlens.shape[0] - 1
    if count_out is None:
        count_out = torch.zeros(1, dtype=torch.int64, device=mask.device)
    _check(_lib.rlf_count_live_responses(_ptr(mask, torch.uint8), _ptr(cu_seqlens, torch.int32), B, T,
                                         _ptr(count_out, torch.int64), _ptr(dev_status, torch.int32), _stream()),
           "rlf_count_live_responses")
    return count_out


def rlf_group_advantage(rewards, group_size=None, group_id=None, num_groups=None, eps=1e-6,
                        unbiased_std=True, adv_out=None, dev_status=None):
    """-> adv fp32[B] on the device."""
    B = rewards.shape[0]
    if adv_out is None:
        adv_out = torch.zeros(B, dtype=torch.float32, device=rewards.device)
    g = int(num_groups) if group_id is not None else int(group_size)
    _check(_lib.rlf_group_advantage(_ptr(rewards, torch.float32), _ptr(group_id, torch.int32), B, g,
                                    float(eps), 1 if unbiased_std else 0, _ptr(adv_out, torch.float32),
                                    _ptr(dev_status, torch.int32), _stream()), "rlf_group_advantage")
    return adv_out


def rlf_rule_reward(scores, weights, reward_out=None):
    """Eq. 1: weighted sum of rule scores.  scores [B, n], weights [n] -> rewards fp32[B]."""
    B, n = scores.shape
    if reward_out is None:
        reward_out = torch.empty(B, dtype=torch.float32, device=scores.device)
    _check(_lib.rlf_rule_reward(_ptr(scores, torch.float32), _ptr(weights, torch.float32), B, n,
                                _ptr(reward_out, torch.float32), _stream()), "rlf_rule_reward")
    return reward_out


KL_K1, KL_K2, KL_K3 = 0, 1, 2


def rlf_kl_in_reward(rewards, old_logp, ref_logp, mask, cu_seqlens, beta, kl_kind=KL_K1, reward_out=None,
                     kl_seq_out=None, dev_status=None):
    """KL penalty folded into the outcome reward: R'_b = R_b - beta * sum_t mask_t k(old_t - ref_t).
    -> (rewards fp32[B], summed estimate per response fp32[B])."""
    B = cu_seqlens.shape[0] - 1
    T = mask.shape[0]
    dev = rewards.device
    if reward_out is None:
        reward_out = torch.empty(B, dtype=torch.float32, device=dev)
    if kl_seq_out is None:
        kl_seq_out = torch.empty(B, dtype=torch.float32, device=dev)
    _check(_lib.rlf_kl_in_reward(_ptr(rewards, torch.float32), _ptr(old_logp, torch.float32),
                                 _ptr(ref_logp, torch.float32), _ptr(mask, torch.uint8),
                                 _ptr(cu_seqlens, torch.int32), B, T, float(beta), int(kl_kind),
                                 _ptr(reward_out, torch.float32), _ptr(kl_seq_out, torch.float32),
                                 _ptr(dev_status, torch.int32), _stream()), "rlf_kl_in_reward")
    return reward_out, kl_seq_out


def rlf_grpo_logp_loss_fwd_bwd(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip, beta_kl,
                               denom=None, grad_logits=None, want_grad=True, in_place=False,
                               logp_out=None, loss_out=None, workspace=None, dev_status=None):
    """logits: [T, V] (rows may be strided, last dim contiguous).
    -> (logp fp32[T], loss fp64[4], grad_logits | None), all on the device."""
    if logits.dim() != 2 or (logits.shape[1] > 1 and logits.stride(1) != 1):
        raise ValueError("logits must be [T, V] with a contiguous last dimension")
    T, V = logits.shape
    stride = logits.stride(0) if T > 1 else max(V, logits.stride(0) if T == 1 else V)
    dev = logits.device
    if grad_logits is None and want_grad:
        grad_logits = logits if in_place else torch.empty_strided((T, V), (stride, 1), dtype=logits.dtype, device=dev)
    if grad_logits is not None and T > 1 and grad_logits.stride(0) != stride:
        raise ValueError("grad_logits must have the row stride of logits")
    if logp_out is None:
        logp_out = torch.empty(T, dtype=torch.float32, device=dev)
    if loss_out is None:
        loss_out = torch.empty(4, dtype=torch.float64, device=dev)
    dt = _dt(logits)
    if workspace is None:
        workspace = new_workspace(FN_LOGP_LOSS, T, V, 0, dt, dev)
    B = adv.shape[0]
    _check(_lib.rlf_grpo_logp_loss_fwd_bwd(
        logits.data_ptr() if T > 0 else None, dt, T, V, stride, _ptr(ids, torch.int32),
        _ptr(seq_id, torch.int32), _ptr(adv, torch.float32), B, _ptr(old_logp, torch.float32),
        _ptr(ref_logp, torch.float32), _ptr(mask, torch.uint8), float(eps_clip), float(beta_kl),
        _ptr(denom, torch.int64), _ptr(logp_out, torch.float32), _ptr(loss_out, torch.float64),
        None if grad_logits is None else grad_logits.data_ptr(), workspace.data_ptr(), workspace.numel(),
        _ptr(dev_status, torch.int32), _stream()), "rlf_grpo_logp_loss_fwd_bwd")
    return logp_out, loss_out, grad_logits


def rlf_grpo_logp_loss_fwd_bwd_obj(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip_low, eps_clip_high,
                                   beta_kl, aggregation=0, denom=None, grad_logits=None, want_grad=True,
                                   in_place=False, logp_out=None, loss_out=None, workspace=None, dev_status=None):
    """Objective variants: asymmetric clip range; aggregation 0 = token mean, 1 = sequence mean."""
    T, V = logits.shape
    stride = logits.stride(0) if T > 1 else V
    dev = logits.device
    if grad_logits is None and want_grad:
        grad_logits = logits if in_place else torch.empty_strided((T, V), (stride, 1), dtype=logits.dtype, device=dev)
    if logp_out is None:
        logp_out = torch.empty(T, dtype=torch.float32, device=dev)
    if loss_out is None:
        loss_out = torch.empty(4, dtype=torch.float64, device=dev)
    dt = _dt(logits)
    if workspace is None:
        workspace = new_workspace(FN_LOGP_LOSS, T, V, 0, dt, dev)
    f = _lib.rlf_grpo_logp_loss_fwd_bwd_obj
    _check(f(logits.data_ptr() if T > 0 else None, dt, T, V, stride, _ptr(ids, torch.int32), _ptr(seq_id, torch.int32),
             _ptr(adv, torch.float32), adv.shape[0], _ptr(old_logp, torch.float32), _ptr(ref_logp, torch.float32),
             _ptr(mask, torch.uint8), float(eps_clip_low), float(eps_clip_high), float(beta_kl), int(aggregation),
             _ptr(denom, torch.int64), _ptr(logp_out, torch.float32), _ptr(loss_out, torch.float64),
             None if grad_logits is None else grad_logits.data_ptr(), workspace.data_ptr(), workspace.numel(),
             _ptr(dev_status, torch.int32), _stream()), "rlf_grpo_logp_loss_fwd_bwd_obj")
    return logp_out, loss_out, grad_logits


def rlf_grpo_logp_loss_fwd_bwd_skip_masked(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip, beta_kl,
                                           denom=None, grad_logits=None, want_grad=True, in_place=False,
                                           zero_masked_grad=True, logp_out=None, loss_out=None, workspace=None,
                                           dev_status=None):
    """As rlf_grpo_logp_loss_fwd_bwd, but rows without loss weight are neither read nor computed."""
    T, V = logits.shape
    stride = logits.stride(0) if T > 1 else V
    dev = logits.device
    if grad_logits is None and want_grad:
        grad_logits = logits if in_place else torch.empty_strided((T, V), (stride, 1), dtype=logits.dtype, device=dev)
    if logp_out is None:
        logp_out = torch.empty(T, dtype=torch.float32, device=dev)
    if loss_out is None:
        loss_out = torch.empty(4, dtype=torch.float64, device=dev)
    dt = _dt(logits)
    if workspace is None:
        workspace = new_workspace(FN_LOGP_LOSS, T, V, 0, dt, dev)
    f = _lib.rlf_grpo_logp_loss_fwd_bwd_skip_masked
    _check(f(logits.data_ptr() if T > 0 else None, dt, T, V, stride, _ptr(ids, torch.int32), _ptr(seq_id, torch.int32),
             _ptr(adv, torch.float32), adv.shape[0], _ptr(old_logp, torch.float32), _ptr(ref_logp, torch.float32),
             _ptr(mask, torch.uint8), float(eps_clip), float(beta_kl), _ptr(denom, torch.int64),
             _ptr(logp_out, torch.float32), _ptr(loss_out, torch.float64),
             None if grad_logits is None else grad_logits.data_ptr(), 1 if zero_masked_grad else 0,
             workspace.data_ptr(), workspace.numel(), _ptr(dev_status, torch.int32), _stream()),
           "rlf_grpo_logp_loss_fwd_bwd_skip_masked")
    return logp_out, loss_out, grad_logits


def rlf_logp_entropy_fwd(logits, ids, want_entropy=True, logp_out=None, entropy_out=None, workspace=None,
                         dev_status=None):
    """Forward only: -> (logp fp32[T], entropy fp32[T] | None) of the rows of `logits` at targets `ids`."""
    T, V = logits.shape
    stride = logits.stride(0) if T > 1 else V
    dev = logits.device
    if logp_out is None:
        logp_out = torch.empty(T, dtype=torch.float32, device=dev)
    if entropy_out is None and want_entropy:
        entropy_out = torch.empty(T, dtype=torch.float32, device=dev)
    dt = _dt(logits)
    if workspace is None:
        workspace = new_workspace(FN_LOGP_ENTROPY, T, V, 0, dt, dev)
    _check(_lib.rlf_logp_entropy_fwd(logits.data_ptr() if T > 0 else None, dt, T, V, stride, _ptr(ids, torch.int32),
                                     _ptr(logp_out, torch.float32), _ptr(entropy_out, torch.float32),
                                     workspace.data_ptr(), workspace.numel(), _ptr(dev_status, torch.int32),
                                     _stream()), "rlf_logp_entropy_fwd")
    return logp_out, entropy_out


STATIC_MAX_TOKENS = 65536


def rlf_grpo_logp_loss_fwd_bwd_static(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip, beta_kl,
                                      denom, logp_out, loss_out, grad_logits=None, dev_status=None):
    """The loss entry point for callers that cannot allocate: no workspace argument (the scratch is a
    fixed array inside the library, at most STATIC_MAX_TOKENS tokens) and, unlike the wrapper above,
    this wrapper creates no tensor either: every output buffer is passed in.  Calls on one device
    share the scratch, so do not let two of them overlap on the GPU."""
    T, V = logits.shape
    stride = logits.stride(0) if T > 1 else V
    _check(_lib.rlf_grpo_logp_loss_fwd_bwd_static(
        logits.data_ptr() if T > 0 else None, _dt(logits), T, V, stride, _ptr(ids, torch.int32),
        _ptr(seq_id, torch.int32), _ptr(adv, torch.float32), adv.shape[0], _ptr(old_logp, torch.float32),
        _ptr(ref_logp, torch.float32), _ptr(mask, torch.uint8), float(eps_clip), float(beta_kl),
        _ptr(denom, torch.int64), _ptr(logp_out, torch.float32), _ptr(loss_out, torch.float64),
        None if grad_logits is None else grad_logits.data_ptr(), _ptr(dev_status, torch.int32), _stream()),
        "rlf_grpo_logp_loss_fwd_bwd_static")
    return logp_out, loss_out, grad_logits


def rlf_fused_lmhead_grpo(hidden, W, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip, beta_kl,
                          denom=None, want_grad_hidden=True, want_grad_W=True, grad_hidden=None, grad_W=None,
                          accumulate_grad_W=False, logp_out=None, loss_out=None, workspace=None,
                          dev_status=None):
    """-> (logp fp32[T], loss fp64[4], grad_hidden bf16[T,D] | None, grad_W fp32[V,D] | None)."""
    T, D = hidden.shape
    V = W.shape[0]
    dev = hidden.device
    if grad_hidden is None and want_grad_hidden:
        grad_hidden = torch.empty((T, D), dtype=torch.bfloat16, device=dev)
    if grad_W is None and want_grad_W:
        grad_W = torch.zeros((V, D), dtype=torch.float32, device=dev)
    if logp_out is None:
        logp_out = torch.empty(T, dtype=torch.float32, device=dev)
    if loss_out is None:
        loss_out = torch.empty(4, dtype=torch.float64, device=dev)
    if workspace is None:
        workspace = new_workspace(FN_FUSED_LMHEAD, T, V, D, RLF_BF16, dev)
    _check(_lib.rlf_fused_lmhead_grpo(
        _ptr(hidden, torch.bfloat16), _ptr(W, torch.bfloat16), T, D, V, _ptr(ids, torch.int32),
        _ptr(seq_id, torch.int32), _ptr(adv, torch.float32), adv.shape[0], _ptr(old_logp, torch.float32),
        _ptr(ref_logp, torch.float32), _ptr(mask, torch.uint8), float(eps_clip), float(beta_kl),
        _ptr(denom, torch.int64), _ptr(logp_out, torch.float32), _ptr(loss_out, torch.float64),
        _ptr(grad_hidden, torch.bfloat16), _ptr(grad_W, torch.float32), 1 if accumulate_grad_W else 0,
        workspace.data_ptr(), workspace.numel(), _ptr(dev_status, torch.int32), _stream()),
        "rlf_fused_lmhead_grpo")
    return logp_out, loss_out, grad_hidden, grad_W


def rlf_fused_lmhead_grpo_obj(hidden, W, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip_low, eps_clip_high,
                              beta_kl, aggregation=0, skip_masked=False, denom=None, want_grad_hidden=True,
                              want_grad_W=True, grad_hidden=None, grad_W=None, accumulate_grad_W=False,
                              logp_out=None, loss_out=None, workspace=None, dev_status=None):
    """The fused LM-head call with an asymmetric clip range, token- or sequence-mean aggregation and
    the option of not multiplying masked rows at all (their log-prob is NaN).
    -> (logp fp32[T], loss fp64[4], grad_hidden bf16[T,D] | None, grad_W fp32[V,D] | None)."""
    T, D = hidden.shape
    V = W.shape[0]
    dev = hidden.device
    if grad_hidden is None and want_grad_hidden:
        grad_hidden = torch.empty((T, D), dtype=torch.bfloat16, device=dev)
    if grad_W is None and want_grad_W:
        grad_W = torch.zeros((V, D), dtype=torch.float32, device=dev)
    if logp_out is None:
        logp_out = torch.empty(T, dtype=torch.float32, device=dev)
    if loss_out is None:
        loss_out = torch.empty(4, dtype=torch.float64, device=dev)
    if workspace is None:
        workspace = new_workspace(FN_FUSED_LMHEAD, T, V, D, RLF_BF16, dev)
    _check(_lib.rlf_fused_lmhead_grpo_obj(
        _ptr(hidden, torch.bfloat16), _ptr(W, torch.bfloat16), T, D, V, _ptr(ids, torch.int32),
        _ptr(seq_id, torch.int32), _ptr(adv, torch.float32), adv.shape[0], _ptr(old_logp, torch.float32),
        _ptr(ref_logp, torch.float32), _ptr(mask, torch.uint8), float(eps_clip_low), float(eps_clip_high),
        float(beta_kl), int(aggregation), 1 if skip_masked else 0, _ptr(denom, torch.int64),
        _ptr(logp_out, torch.float32), _ptr(loss_out, torch.float64), _ptr(grad_hidden, torch.bfloat16),
        _ptr(grad_W, torch.float32), 1 if accumulate_grad_W else 0, workspace.data_ptr(), workspace.numel(),
        _ptr(dev_status, torch.int32), _stream()), "rlf_fused_lmhead_grpo_obj")
    return logp_out, loss_out, grad_hidden, grad_W


def rlf_fused_lmhead_logp_entropy(hidden, W, ids, want_entropy=True, logp_out=None, entropy_out=None,
                                  workspace=None, dev_status=None):
    """Forward only, from hidden states: -> (logp fp32[T], entropy fp32[T] | None); logits are never stored."""
    T, D = hidden.shape
    V = W.shape[0]
    dev = hidden.device
    if logp_out is None:
        logp_out = torch.empty(T, dtype=torch.float32, device=dev)
    if entropy_out is None and want_entropy:
        entropy_out = torch.empty(T, dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = new_workspace(FN_FUSED_LOGP_ENTROPY, T, V, D, RLF_BF16, dev)
    _check(_lib.rlf_fused_lmhead_logp_entropy(
        _ptr(hidden, torch.bfloat16) if T > 0 else None, _ptr(W, torch.bfloat16), T, D, V, _ptr(ids, torch.int32),
        _ptr(logp_out, torch.float32), _ptr(entropy_out, torch.float32), workspace.data_ptr(), workspace.numel(),
        _ptr(dev_status, torch.int32), _stream()), "rlf_fused_lmhead_logp_entropy")
    return logp_out, entropy_out


def step_arena_bytes(T, V, B, dt=RLF_BF16):
    return int(_lib.rlf_step_arena_bytes(T, V, B, dt))


def rlf_grpo_step_host(h_logits, h_ids, h_cu_seqlens, group_size, h_rewards, h_old_logp, h_ref_logp,
                       open_id, close_id, adv_eps, eps_clip, beta_kl, h_loss_out, d_arena, h_logp_out=None,
                       h_mask_out=None, h_dev_status=None):
    """One whole step from host tensors (pinned for full copy rate); waits for completion."""
    T, V = h_logits.shape
    B = h_rewards.shape[0]
    _check(_lib.rlf_grpo_step_host(
        _ptr(h_logits, cuda=False), _dt(h_logits), T, V, _ptr(h_ids, torch.int32, False),
        _ptr(h_cu_seqlens, torch.int32, False), B, int(group_size), _ptr(h_rewards, torch.float32, False),
        _ptr(h_old_logp, torch.float32, False), _ptr(h_ref_logp, torch.float32, False), open_id, close_id,
        float(adv_eps), float(eps_clip), float(beta_kl), _ptr(h_loss_out, torch.float64, False),
        _ptr(h_logp_out, torch.float32, False), _ptr(h_mask_out, torch.uint8, False),
        _ptr(h_dev_status, torch.int32, False), d_arena.data_ptr(), d_arena.numel(), _stream()),
        "rlf_grpo_step_host")
    return h_loss_out
