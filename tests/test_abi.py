"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, and
its host-side argument validation answers before any device work (no compute without a GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2509_06980_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "rlf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rlf_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_path_entry_points():
    syms = _declared_symbols()
    for name in ("rlf_build_loss_mask", "rlf_group_advantage", "rlf_grpo_logp_loss_fwd_bwd",
                 "rlf_fused_lmhead_grpo"):
        assert name in syms


def test_library_exports_every_declared_symbol(lib):
    for name in _declared_symbols():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2509_06980_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_symbols()


def test_status_strings_and_version(lib):
    lib.rlf_status_string.restype = ctypes.c_char_p
    seen = set()
    for code in range(0, -10, -1):           # RLF_OK .. RLF_ERR_TOO_LARGE (-9)
        s = lib.rlf_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 10
    assert "RLF_STATIC_MAX_TOKENS" in lib.rlf_status_string(-9).decode()
    assert lib.rlf_status_string(-99).decode() == "unknown status"
    assert lib.rlf_version() >= 100


def test_workspace_sizes(lib):
    lib.rlf_workspace_bytes.restype = ctypes.c_size_t
    lib.rlf_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int]
    small = lib.rlf_workspace_bytes(3, 0, 1024, 0, 0)
    big = lib.rlf_workspace_bytes(3, 32768, 151936, 0, 0)
    assert small > 0 and big >= small + 16 * 32768
    assert lib.rlf_workspace_bytes(99, 10, 10, 10, 0) == 0


def test_host_validation_rejects_bad_arguments_before_touching_a_device(lib):
    vp = ctypes.c_void_p
    f = lib.rlf_grpo_logp_loss_fwd_bwd
    f.argtypes = [vp, ctypes.c_int, ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, vp, vp, vp, ctypes.c_int32,
                  vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, vp, vp, vp, vp, ctypes.c_size_t, vp, vp]
    fake = 4096  # never dereferenced: every case fails validation first
    args = lambda **kw: [kw.get("logits", fake), kw.get("dt", 0), kw.get("T", 4), kw.get("V", 64),
                         kw.get("stride", 64), fake, fake, fake, kw.get("B", 1), fake, fake, fake, 0.2, 0.001,
                         None, fake, kw.get("loss", fake), None, kw.get("ws", fake), kw.get("wsb", 1 << 30),
                         None, None]
    assert f(*args(dt=7)) == -4
    assert f(*args(T=-1)) == -2
    assert f(*args(V=0)) == -2
    assert f(*args(stride=8)) == -2
    assert f(*args(loss=None)) == -1
    assert f(*args(logits=None)) == -1
    assert f(*args(logits=4097)) == -3
    assert f(*args(ws=None)) == -5
    assert f(*args(ws=4100)) == -5
    assert f(*args(wsb=16)) == -5
    g = lib.rlf_build_loss_mask
    g.argtypes = [vp, vp, ctypes.c_int32, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, vp, vp, vp, vp, vp, vp]
    assert g(fake, fake, -1, 4, 1, 2, None, fake, None, fake, None, None) == -2
    assert g(fake, fake, 1, 4, 1, 2, None, fake, None, None, None, None) == -1
    assert g(None, fake, 1, 4, 1, 2, None, fake, None, fake, None, None) == -1
    h = lib.rlf_group_advantage
    h.argtypes = [vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_float, ctypes.c_int, vp, vp, vp]
    assert h(fake, None, 4, 0, 1e-6, 1, fake, None, None) == -2
    assert h(None, None, 4, 2, 1e-6, 1, fake, None, None) == -1
    assert h(fake, None, 0, 2, 1e-6, 1, fake, None, None) == 0
    k = lib.rlf_kl_in_reward
    k.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_int, vp, vp, vp, vp]
    assert k(fake, fake, fake, fake, fake, 2, 8, 0.1, 5, fake, None, None, None) == -8
    assert k(fake, fake, fake, fake, fake, -1, 8, 0.1, 0, fake, None, None, None) == -2
    assert k(fake, fake, fake, fake, None, 2, 8, 0.1, 0, fake, None, None, None) == -1
    assert k(fake, None, fake, fake, fake, 2, 8, 0.1, 0, fake, None, None, None) == -1
    assert k(fake, fake, fake, fake, fake, 0, 8, 0.1, 0, fake, None, None, None) == 0
    e = lib.rlf_fused_lmhead_logp_entropy
    e.argtypes = [vp, vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, vp, vp, vp, vp, ctypes.c_size_t, vp, vp]
    assert e(fake, fake, 8, 100, 64, fake, fake, None, fake, 1 << 30, None, None) == -2      # D not a multiple of 64
    assert e(fake, fake, 8, 128, 63, fake, fake, None, fake, 1 << 30, None, None) == -2      # V not a multiple of 8
    assert e(None, fake, 8, 128, 64, fake, fake, None, fake, 1 << 30, None, None) == -1
    assert e(fake, fake, 8, 128, 64, fake, None, None, fake, 1 << 30, None, None) == -1
    assert e(4104, fake, 8, 128, 64, fake, fake, None, fake, 1 << 30, None, None) == -3      # hidden not 16-byte aligned
    assert e(fake, fake, 8, 128, 64, fake, fake, None, fake, 16, None, None) == -5
    assert e(fake, fake, 0, 128, 64, None, None, None, None, 0, None, None) == 0             # T = 0: nothing to do
    o = lib.rlf_fused_lmhead_grpo_obj
    o.argtypes = [vp, vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, vp, vp, vp, ctypes.c_int32, vp, vp, vp,
                  ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp,
                  ctypes.c_int, vp, ctypes.c_size_t, vp, vp]
    oargs = lambda agg=0, skip=0, B=1: [fake, fake, 8, 128, 64, fake, fake, fake, B, fake, fake, fake, 0.2, 0.3, 0.0, agg,
                                        skip, None, fake, fake, None, None, 0, fake, 1 << 30, None, None]
    assert o(*oargs(agg=2)) == -2 and o(*oargs(skip=2)) == -2 and o(*oargs(agg=1, B=100)) == -2
    s = lib.rlf_tune_lmhead_schedule
    s.argtypes = [ctypes.c_int] * 3
    assert s(-1, 0, 0) == -2 and s(0, -1, 0) == -2 and s(0, 0, 3) == -2 and s(0, 0, 0) == 0
    bw = lib.rlf_tune_lmhead_backward
    bw.argtypes = [ctypes.c_int] * 2
    assert bw(2, 1) == -2 and bw(1, -1) == -2 and bw(0, 0) == 0 and bw(1, 1) == 0
    pc = lib.rlf_tune_lmhead_pacing
    pc.argtypes = [ctypes.c_int]
    assert pc(2) == -2 and pc(-1) == -2 and pc(0) == 0 and pc(1) == 0
    t = lib.rlf_tune_logits_kernel
    t.argtypes = [ctypes.c_int] * 3
    assert t(17, 256, 0) == -2 and t(-1, 256, 0) == -2 and t(4, 500, 0) == -2 and t(3, 512, 0) == 0 and t(0, 0, -1) == 0


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2509_06980_b200")
    pat = re.compile(r"(import\s+oracle|from\s+oracle|rlf_oracle|orc_[a-z_]+\s*\(|oracle/)")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert not pat.search(text), fn
