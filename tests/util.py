"""Helpers shared by the tests (no method arithmetic: fixtures parsing and error metrics)."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            rows.append([c.strip() for c in line.split("|")])
    return rows


def bf16_ulp(x):
    """Unit in the last place of bfloat16 (8 significand bits) at the binade of |x| (fp64 array).
    Below the smallest normal the subnormal spacing 2^-133 is used."""
    ax = np.abs(np.asarray(x, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(ax, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def ulp_error_bf16(got_f64, want_f64):
    """|got - want| in bf16 ulps of `want`; values of `want` below the smallest bf16 normal
    count as matching zero or any subnormal."""
    got = np.asarray(got_f64, np.float64)
    want = np.asarray(want_f64, np.float64)
    err = np.abs(got - want) / bf16_ulp(want)
    tiny = (np.abs(want) < 2.0 ** -126) & (np.abs(got) < 2.0 ** -126)
    return np.where(tiny, 0.0, err)


def loss_close(got, want, scale_floor, rel=1e-4):
    """Scalar-loss criterion: |got - want| <= rel * max(|want|, scale_floor)."""
    return abs(got - want) <= rel * max(abs(want), scale_floor)
