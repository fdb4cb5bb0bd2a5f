"""ctypes front end of the fp64 CPU oracle (oracle/rlf_oracle.c).

TEST INFRASTRUCTURE ONLY.  This module marshals numpy arrays into the C
functions and holds no arithmetic of its own.  It never imports the CUDA
package, and the CUDA package never imports it.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rlf_oracle.c")
_LIB = os.path.join(_HERE, "librlf_oracle.so")

BF16, F32, F64 = 0, 1, 2

_lib = None


def build(force=False):
    """Compile the oracle with gcc (OpenMP over independent rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    """The compiled oracle.  RLF_ORACLE_LIB names another build of it (used by the mutation tests,
    which check that the pins notice a planted mistake)."""
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(os.environ.get("RLF_ORACLE_LIB") or build())
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dt):
    if a is None:
        return None
    return np.ascontiguousarray(a, dtype=dt)


def _check(rc, what):
    if rc != 0:
        raise ValueError("%s: oracle returned %d" % (what, rc))


def num_threads():
    return int(lib().orc_num_threads())


def build_loss_mask(ids, cu_seqlens, open_id, close_id, valid=None):
    """-> (mask u8[T], seq_id i32[T], N int)."""
    ids = _c(ids, np.int32)
    cu = _c(cu_seqlens, np.int32)
    valid = _c(valid, np.uint8)
    T = ids.shape[0]
    B = cu.shape[0] - 1
    mask = np.empty(T, np.uint8)
    seq = np.empty(T, np.int32)
    n = ctypes.c_int64(0)
    rc = lib().orc_build_loss_mask(_p(ids), _p(cu), ctypes.c_int32(B), ctypes.c_int64(T),
                                   ctypes.c_int32(open_id), ctypes.c_int32(close_id), _p(valid),
                                   _p(mask), _p(seq), ctypes.byref(n))
    _check(rc, "build_loss_mask")
    return mask, seq, int(n.value)


def group_advantage(rewards, group_id=None, group_size=None, num_groups=None, eps=1e-6,
                    unbiased=True):
    """-> adv f64[B]."""
    r = _c(rewards, np.float32)
    B = r.shape[0]
    gid = _c(group_id, np.int32)
    g = int(num_groups) if gid is not None else int(group_size)
    adv = np.zeros(B, np.float64)
    rc = lib().orc_group_advantage(_p(r), _p(gid), ctypes.c_int32(B), ctypes.c_int32(g),
                                   ctypes.c_double(eps), ctypes.c_int(1 if unbiased else 0), _p(adv))
    _check(rc, "group_advantage")
    return adv


def _dtype_code(a):
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float64:
        return F64
    raise TypeError("logits must be uint16 (bf16 bits), float32 or float64")


def grpo_loss(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip, beta_kl,
              denom=None, want_grad=True, want_coef=False):
    """logits: 2-D numpy array, dtype uint16 (bf16 bit patterns), float32 or float64;
    rows may be strided (last dim contiguous).
    -> dict(logp f64[T], loss f64[4], grad f64[T,V] | None, coef f64[T] | None)."""
    assert logits.ndim == 2 and (logits.shape[1] <= 1 or logits.strides[1] == logits.itemsize)
    T, V = logits.shape
    stride = logits.strides[0] // logits.itemsize if T > 1 else V
    ids = _c(ids, np.int32)
    seq_id = _c(seq_id, np.int32)
    adv = _c(adv, np.float32)
    old_logp = _c(old_logp, np.float32)
    ref_logp = _c(ref_logp, np.float32)
    mask = _c(mask, np.uint8)
    logp = np.zeros(T, np.float64)
    loss = np.zeros(4, np.float64)
    grad = np.zeros((T, V), np.float64) if want_grad else None
    coef = np.zeros(T, np.float64) if want_coef else None
    rc = lib().orc_grpo_loss(_p(logits), ctypes.c_int(_dtype_code(logits)), ctypes.c_int64(T),
                             ctypes.c_int32(V), ctypes.c_int64(stride), _p(ids), _p(seq_id), _p(adv),
                             _p(old_logp), _p(ref_logp), _p(mask), ctypes.c_double(eps_clip),
                             ctypes.c_double(beta_kl),
                             ctypes.c_int64(-1 if denom is None else int(denom)),
                             _p(logp), _p(loss), _p(grad), _p(coef))
    _check(rc, "grpo_loss")
    return dict(logp=logp, loss=loss, grad=grad, coef=coef)


def grpo_loss_obj(logits, ids, seq_id, adv, old_logp, ref_logp, mask, eps_low, eps_high, beta_kl, aggregation=0,
                  denom=None, want_grad=True, want_coef=False):
    """Objective variants: asymmetric clip range and token-mean (0) / sequence-mean (1) aggregation.
    -> dict(logp, loss f64[4], grad | None, coef | None)."""
    assert logits.ndim == 2 and (logits.shape[1] <= 1 or logits.strides[1] == logits.itemsize)
    T, V = logits.shape
    stride = logits.strides[0] // logits.itemsize if T > 1 else V
    ids = _c(ids, np.int32)
    seq_id = _c(seq_id, np.int32)
    adv = _c(adv, np.float32)
    old_logp = _c(old_logp, np.float32)
    ref_logp = _c(ref_logp, np.float32)
    mask = _c(mask, np.uint8)
    logp = np.zeros(T, np.float64)
    loss = np.zeros(4, np.float64)
    grad = np.zeros((T, V), np.float64) if want_grad else None
    coef = np.zeros(T, np.float64) if want_coef else None
    rc = lib().orc_grpo_loss_obj(_p(logits), ctypes.c_int(_dtype_code(logits)), ctypes.c_int64(T), ctypes.c_int32(V),
                                 ctypes.c_int64(stride), _p(ids), _p(seq_id), _p(adv), ctypes.c_int32(adv.shape[0]),
                                 _p(old_logp), _p(ref_logp), _p(mask), ctypes.c_double(eps_low),
                                 ctypes.c_double(eps_high), ctypes.c_double(beta_kl), ctypes.c_int(aggregation),
                                 ctypes.c_int64(-1 if denom is None else int(denom)), _p(logp), _p(loss), _p(grad),
                                 _p(coef))
    _check(rc, "grpo_loss_obj")
    return dict(logp=logp, loss=loss, grad=grad, coef=coef)


def logp_entropy(logits, ids, want_entropy=True):
    """-> (logp f64[T], entropy f64[T] | None) of each row's softmax at the given targets."""
    assert logits.ndim == 2 and (logits.shape[1] <= 1 or logits.strides[1] == logits.itemsize)
    T, V = logits.shape
    stride = logits.strides[0] // logits.itemsize if T > 1 else V
    ids = _c(ids, np.int32)
    logp = np.zeros(T, np.float64)
    ent = np.zeros(T, np.float64) if want_entropy else None
    rc = lib().orc_logp_entropy(_p(logits), ctypes.c_int(_dtype_code(logits)), ctypes.c_int64(T), ctypes.c_int32(V),
                                ctypes.c_int64(stride), _p(ids), _p(logp), _p(ent))
    _check(rc, "logp_entropy")
    return logp, ent


def fused_lmhead_grpo(hidden, W, ids, seq_id, adv, old_logp, ref_logp, mask, eps_clip, beta_kl,
                      denom=None, want_grad_hidden=True, want_grad_W=True, want_z=False):
    """hidden [T,D], W [V,D]: uint16 arrays holding bf16 bit patterns.
    -> dict(logp, loss, grad_hidden f64[T,D] | None, grad_W f64[V,D] | None, z f64[T,V] | None)."""
    hidden = _c(hidden, np.uint16)
    W = _c(W, np.uint16)
    T, D = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == D
    ids = _c(ids, np.int32)
    seq_id = _c(seq_id, np.int32)
    adv = _c(adv, np.float32)
    old_logp = _c(old_logp, np.float32)
    ref_logp = _c(ref_logp, np.float32)
    mask = _c(mask, np.uint8)
    logp = np.zeros(T, np.float64)
    loss = np.zeros(4, np.float64)
    gh = np.zeros((T, D), np.float64) if want_grad_hidden else None
    gw = np.zeros((V, D), np.float64) if want_grad_W else None
    z = np.zeros((T, V), np.float64) if want_z else None
    rc = lib().orc_fused_lmhead_grpo(_p(hidden), _p(W), ctypes.c_int64(T), ctypes.c_int32(D),
                                     ctypes.c_int32(V), _p(ids), _p(seq_id), _p(adv), _p(old_logp),
                                     _p(ref_logp), _p(mask), ctypes.c_double(eps_clip),
                                     ctypes.c_double(beta_kl),
                                     ctypes.c_int64(-1 if denom is None else int(denom)),
                                     _p(logp), _p(loss), _p(gh), _p(gw), _p(z))
    _check(rc, "fused_lmhead_grpo")
    return dict(logp=logp, loss=loss, grad_hidden=gh, grad_W=gw, z=z)


def rule_reward(scores, weights):
    """Eq. 1: weighted sum of rule scores.  scores [B,n], weights [n] -> R f64[B]."""
    s = _c(scores, np.float32)
    w = _c(weights, np.float32)
    B, n = s.shape
    R = np.zeros(B, np.float64)
    rc = lib().orc_rule_reward(_p(s), _p(w), ctypes.c_int32(B), ctypes.c_int32(n), _p(R))
    _check(rc, "rule_reward")
    return R


def kl_in_reward(rewards, old_logp, ref_logp, mask, cu_seqlens, beta, kind=0):
    """KL penalty folded into the outcome reward.  -> (R' f64[B], kl_seq f64[B])."""
    r = _c(rewards, np.float32)
    old_logp = _c(old_logp, np.float32)
    ref_logp = _c(ref_logp, np.float32)
    mask = _c(mask, np.uint8)
    cu = _c(cu_seqlens, np.int32)
    B = len(cu) - 1
    T = len(mask)
    out = np.zeros(B, np.float64)
    kl = np.zeros(B, np.float64)
    rc = lib().orc_kl_in_reward(_p(r), _p(old_logp), _p(ref_logp), _p(mask), _p(cu), ctypes.c_int32(B),
                                ctypes.c_int64(T), ctypes.c_double(beta), ctypes.c_int(kind), _p(out), _p(kl))
    _check(rc, "kl_in_reward")
    return out, kl


def fused_lmhead_grpo_obj(hidden, W, ids, seq_id, adv, old_logp, ref_logp, mask, eps_low, eps_high, beta_kl,
                          aggregation=0, denom=None, want_grad_hidden=True, want_grad_W=True):
    """The fused LM-head variant under the objective variants.  hidden [T,D], W [V,D]: bf16 bit patterns.
    -> dict(logp, loss, grad_hidden f64[T,D] | None, grad_W f64[V,D] | None)."""
    hidden = _c(hidden, np.uint16)
    W = _c(W, np.uint16)
    T, D = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == D
    ids = _c(ids, np.int32)
    seq_id = _c(seq_id, np.int32)
    adv = _c(adv, np.float32)
    old_logp = _c(old_logp, np.float32)
    ref_logp = _c(ref_logp, np.float32)
    mask = _c(mask, np.uint8)
    logp = np.zeros(T, np.float64)
    loss = np.zeros(4, np.float64)
    gh = np.zeros((T, D), np.float64) if want_grad_hidden else None
    gw = np.zeros((V, D), np.float64) if want_grad_W else None
    rc = lib().orc_fused_lmhead_grpo_obj(_p(hidden), _p(W), ctypes.c_int64(T), ctypes.c_int32(D), ctypes.c_int32(V),
                                         _p(ids), _p(seq_id), _p(adv), ctypes.c_int32(len(adv)), _p(old_logp),
                                         _p(ref_logp), _p(mask), ctypes.c_double(eps_low), ctypes.c_double(eps_high),
                                         ctypes.c_double(beta_kl), ctypes.c_int(aggregation),
                                         ctypes.c_int64(-1 if denom is None else int(denom)), _p(logp), _p(loss),
                                         _p(gh), _p(gw))
    _check(rc, "fused_lmhead_grpo_obj")
    return dict(logp=logp, loss=loss, grad_hidden=gh, grad_W=gw)


def fused_lmhead_logp_entropy(hidden, W, ids, want_entropy=True):
    """hidden [T,D], W [V,D]: bf16 bit patterns -> (logp f64[T], entropy f64[T] | None)."""
    hidden = _c(hidden, np.uint16)
    W = _c(W, np.uint16)
    T, D = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == D
    ids = _c(ids, np.int32)
    logp = np.zeros(T, np.float64)
    ent = np.zeros(T, np.float64) if want_entropy else None
    rc = lib().orc_fused_lmhead_logp_entropy(_p(hidden), _p(W), ctypes.c_int64(T), ctypes.c_int32(D),
                                             ctypes.c_int32(V), _p(ids), _p(logp), _p(ent))
    _check(rc, "fused_lmhead_logp_entropy")
    return logp, ent
