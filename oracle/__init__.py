"""CPU oracle for the STEP hot path (decode attention, step scorer, prune) and what was built around it.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, obviously-correct
restatement of what the method computes, written from the paper's equations
and Algorithm 1.  It shares no code with the CUDA path and imports nothing
from it; the product never routes through it.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it.

Contents
--------
attention.py  softmax(q K^T / sqrt(d)) V per trace over its logical token
              sequence, dense and through a block table (fp64).
scorer.py     step scorer y = sigmoid(W2 ReLU(W1 h + b1) + b2) (Sec. 3.1,
              "Model Architecture") and the running-mean trace score
              (Sec. 3.3, running-average equation).
kv_pool.py    paged KV pool bookkeeping: InitTraces prefix fork, append,
              the memory trigger and the evict-lowest-score rule of
              Algorithm 1 / Sec. 3.2, block reclaim; the weighted vote.
steps.py      step-end test of a sampled token's text (Sec. 3.1 footnote).
algorithm1.py the loop of Algorithm 1 over the pieces above.
training.py   weighted BCE-from-logits loss, its gradients and Adam for the
              scorer (Sec. 3.1 "Training Objective"; appendix parameters).

Every function is pinned by tests that do not re-use its own formula
(brute force on unpaged data, closed forms, hand-worked examples,
invariants); nothing here is "parity unpinned".
"""
