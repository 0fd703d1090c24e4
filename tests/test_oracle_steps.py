"""Pins for the step-end oracle and the library's host-side vocabulary table (no GPU needed)."""
import ast
import os

import numpy as np

from oracle import steps as OSt
from paper_2601_09093_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "step_end_examples.txt")


def _examples():
    out = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        text, flag = line.rstrip("\n").split("\t")
        out.append((ast.literal_eval(text), int(flag)))
    return out


def test_golden_examples():
    ex = _examples()
    assert len(ex) >= 10
    for text, flag in ex:
        assert OSt.is_step_end(text) == bool(flag), text
        assert OSt.is_step_end(text.decode()) == bool(flag)


def test_agrees_with_splitting_the_text_at_the_delimiter():
    """A token contains the delimiter exactly when cutting its text at the delimiter yields more than one piece
    (the paper's segmentation of the reasoning text, applied to a single token)."""
    vocab = W.synthetic_vocab(7, 4000, step_end_frac=0.05)
    for t in vocab:
        assert OSt.is_step_end(t) == (len(t.split(b"\n\n")) > 1)
    n = sum(OSt.is_step_end(t) for t in vocab)
    assert 100 < n < 600                                  # planted ones plus a few by chance


def test_mask_over_sampled_tokens_brute_force():
    vocab = W.synthetic_vocab(3, 500, step_end_frac=0.1)
    ends = [v for v, t in enumerate(vocab) if b"\n\n" in t]
    ids = W.token_ids(3, 1000, len(vocab), ends, density=0.2)
    ids[5], ids[6] = -1, len(vocab)                       # outside the vocabulary: never a step end
    m = OSt.step_end_mask(ids, vocab)
    for i, t in enumerate(ids):
        want = 0 <= t < len(vocab) and vocab[t].find(b"\n\n") >= 0
        assert m[i] == int(want)
    assert m[5] == 0 and m[6] == 0 and 150 < m.sum() < 350


def test_library_host_table_matches_the_oracle():
    from paper_2601_09093_b200 import binding as B
    vocab = W.synthetic_vocab(11, 3000, step_end_frac=0.02) + [t for t, _ in _examples()] + [None]
    table = B.step_end_table_from_vocab(vocab).numpy()
    want = np.array([OSt.is_step_end(t) for t in vocab], dtype=np.uint8)
    np.testing.assert_array_equal(table, want)
