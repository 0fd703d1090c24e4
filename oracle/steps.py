"""Oracle: step-end detection (fp-free; plain string search).

TEST INFRASTRUCTURE ONLY - never imported by the product path.

Sec. 3.1 "Step Representation": the reasoning text is cut into steps at the delimiter made of two newline
characters in a row, and the step-end token is, by the paper's footnote, any token whose text contains that
delimiter.  Algorithm 1 applies exactly this test to each sampled token x before calling the scorer.
"""
from __future__ import annotations

import numpy as np

DELIMITER = b"\n\n"


def is_step_end(token_text) -> bool:
    """True iff the token's text contains the step delimiter."""
    if token_text is None:
        return False
    if isinstance(token_text, str):
        token_text = token_text.encode("utf-8")
    return DELIMITER in token_text


def step_end_mask(token_ids, vocab_texts) -> np.ndarray:
    """mask[i] = 1 iff the text of sampled token i ends a step; an id outside the vocabulary ends none."""
    out = np.zeros(len(token_ids), dtype=np.uint8)
    for i, t in enumerate(token_ids):
        t = int(t)
        if 0 <= t < len(vocab_texts) and is_step_end(vocab_texts[t]):
            out[i] = 1
    return out
