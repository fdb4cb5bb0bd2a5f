"""Pins for the oracle's loss mask (Sec. 2.2 / Sec. 2.3.2: observation tokens carry no loss)."""
import numpy as np
import pytest

from oracle import rlf_oracle as orc
from paper_2509_06980_b200 import synth
from util import read_golden

O, C = synth.OPEN_ID, synth.CLOSE_ID


def _encode(s):
    """'xox/xc' -> ids, cu_seqlens."""
    ids, cu = [], [0]
    filler = 7
    for seq in s.split("/"):
        for ch in seq:
            ids.append({"o": O, "c": C, "x": filler}[ch])
            filler = filler + 1 if filler < 900 else 7
        cu.append(len(ids))
    return np.array(ids, np.int32), np.array(cu, np.int32)


@pytest.mark.parametrize("name,toks,want", read_golden("mask_cases.txt"))
def test_hand_cases(name, toks, want):
    ids, cu = _encode(toks)
    mask, seq, n = orc.build_loss_mask(ids, cu, O, C)
    want_bits = [int(ch) for ch in want.replace("/", "")]
    assert mask.tolist() == want_bits, name
    assert n == sum(want_bits)
    want_seq = [b for b, seq_s in enumerate(toks.split("/")) for _ in seq_s]
    assert seq.tolist() == want_seq


def _last_marker_rule(ids, cu):
    """Independent formulation: a token is excluded iff it is an open marker, or the nearest
    marker strictly before it in its own sequence is an open marker."""
    mask = np.zeros(len(ids), np.uint8)
    for b in range(len(cu) - 1):
        for t in range(cu[b], cu[b + 1]):
            prev = [u for u in range(cu[b], t) if ids[u] in (O, C)]
            inside_before = bool(prev) and ids[prev[-1]] == O
            mask[t] = 0 if (ids[t] == O or inside_before) else 1
    return mask


def test_brute_force_random_streams():
    rng = np.random.default_rng(7)
    for trial in range(200):
        B = int(rng.integers(1, 5))
        lens = rng.integers(0, 40, size=B)
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        T = int(cu[-1])
        # dense markers so that nested opens, stray closes and unclosed spans all occur
        ids = rng.choice([O, C, 5, 6, 7], size=T, p=[0.2, 0.2, 0.2, 0.2, 0.2]).astype(np.int32)
        mask, seq, n = orc.build_loss_mask(ids, cu, O, C)
        assert mask.tolist() == _last_marker_rule(ids, cu).tolist()
        assert n == int(mask.sum())


@pytest.mark.parametrize("cfg", [0, 1, 2, 4])
def test_count_identity_on_generated_streams(cfg):
    """The generator places disjoint spans of known total length: N = T - (obs + markers)."""
    tok = synth.make_tokens(synth.SPECS[cfg])
    mask, seq, n = orc.build_loss_mask(tok.ids, tok.cu_seqlens, O, C)
    T = len(tok.ids)
    assert n == T - tok.n_span_tokens
    for (b, s, k) in tok.spans[:50]:
        a = tok.cu_seqlens[b] + s
        assert not mask[a:a + k + 2].any()
        assert mask[a - 1] == 1 and mask[a + k + 2] == 1
    assert (np.diff(seq) >= 0).all() and seq[0] == 0 and seq[-1] == len(tok.cu_seqlens) - 2


def test_concatenation_independence():
    """Masks of concatenated sequences are the concatenated masks."""
    rng = np.random.default_rng(11)
    parts = [rng.choice([O, C, 3, 4], size=int(rng.integers(1, 30))).astype(np.int32) for _ in range(6)]
    singles = [orc.build_loss_mask(p, np.array([0, len(p)], np.int32), O, C)[0] for p in parts]
    cu = np.concatenate([[0], np.cumsum([len(p) for p in parts])]).astype(np.int32)
    joint = orc.build_loss_mask(np.concatenate(parts), cu, O, C)[0]
    assert joint.tolist() == np.concatenate(singles).tolist()


def test_valid_mask_is_anded():
    ids, cu = _encode("xxoxcxx")
    valid = np.array([1, 0, 1, 1, 1, 0, 1], np.uint8)
    mask, _, n = orc.build_loss_mask(ids, cu, O, C, valid)
    assert mask.tolist() == [1, 0, 0, 0, 0, 0, 1] and n == 2


def test_empty():
    mask, seq, n = orc.build_loss_mask(np.zeros(0, np.int32), np.array([0], np.int32), O, C)
    assert len(mask) == 0 and n == 0
