"""Pins for the Algorithm 1 oracle: the example worked by hand in tests/golden, and structural properties."""
import math
import os

import numpy as np

from oracle.algorithm1 import Algorithm1Oracle
from oracle.kv_pool import KVPoolOracle
from paper_2601_09093_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "algorithm1_hand_example.txt")
VOCAB = [b"a", b"\n\n", b"<eos>"]


def _h(tok):
    return {"ln9": math.log(9.0), "ln3": math.log(3.0), "0": 0.0}[tok]


def load_hand_example():
    rows, answers, vote = [], None, None
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        parts = [p.strip() for p in line.split("|")]
        if parts[0] == "answers":
            answers = [int(x) for x in parts[1].split()]
        elif parts[0] == "vote":
            vote = int(parts[1])
        else:
            ids = lambda s: [] if s == "-" else [int(x) for x in s.split()]
            rows.append(dict(tokens=[int(x) for x in parts[1].split()], h=[_h(x) for x in parts[2].split()],
                             evicted=ids(parts[3]), finished=ids(parts[4]), used=int(parts[5]),
                             scores=[None if x == "-" else float(x) for x in parts[6].split()]))
    return rows, answers, vote


def make_hand_oracle():
    pool = KVPoolOracle(1, 1, 1, 2, 6, 3, 8, store_payload=False)
    pool.fork_prefix(3, 2)
    return Algorithm1Oracle(pool, 3, np.ones((1, 1)), np.zeros(1), np.ones(1), 0.0, VOCAB, 2, 1.0, -1.0)


def test_hand_worked_example():
    rows, answers, vote = load_hand_example()
    o = make_hand_oracle()
    for r in rows:
        live_before = o.live()
        scores_at_scoring = {}
        ev = o.iteration(np.array(r["tokens"]), np.array(r["h"]).reshape(3, 1), answers)
        assert ev["evicted"] == r["evicted"] and ev["finished"] == r["finished"]
        assert o.pool.used == r["used"]
        for t, want in enumerate(r["scores"]):
            if want is None:
                assert t not in live_before
            elif t in o.finished:
                assert abs(o.finished[t][0] - want) < 1e-12
            elif o.pool.live[t]:
                assert abs(o.ts.score(t) - want) < 1e-12
        o.pool.check_invariants()
    assert o.live() == [] and o.n_evicted == 1
    assert o.vote() == vote
    assert {t: a for t, (_, a) in o.finished.items()} == {2: 42, 0: 7}


def _random_run(seed, n=12, keep_frac=-1.0, threshold=1.0, iters=400, max_evictions=4):
    cfg = W.scaled(W.C0, scorer_D=16, scorer_m=8, seed=seed)
    vocab = W.synthetic_vocab(seed, 200, step_end_frac=0.1)
    eos = 0
    ends = [v for v, t in enumerate(vocab) if b"\n\n" in t]
    g = W.rng(seed, W.TID_TOK, 99)
    toks = np.stack([W.token_ids(seed, n, len(vocab), ends, 0.2, sub=i) for i in range(iters)])
    toks[toks == eos] = 1
    toks[g.random(toks.shape) < 0.02] = eos                      # ~2 % chance per step that a trace completes
    toks[iters - 1] = eos
    (_, W1), (_, b1), (_, w2), b2 = W.scorer_weights(cfg, std=0.5, bias_std=0.1)
    _, hid = W.normal(seed, W.TID_HID, (iters, n, 16), "fp32")
    answers = W.rng(seed, W.TID_ANS).integers(0, 4, size=n)
    pool = KVPoolOracle(1, 1, 4, 4, 30, n, 64, store_payload=False)
    pool.fork_prefix(n, 8)
    o = Algorithm1Oracle(pool, n, W1, b1, w2, b2, vocab, eos, threshold, keep_frac, max_evictions=max_evictions)
    return o, toks, hid, answers


def test_every_trace_completes_or_is_evicted_and_all_kv_returns():
    for seed in (1, 2, 3):
        o, toks, hid, answers = _random_run(seed)
        ans, log = o.run(toks, hid, answers)
        evicted = [t for e in log for t in e["evicted"]]
        done = [t for e in log for t in e["finished"]]
        assert sorted(evicted + done) == list(range(12)) and o.live() == []
        assert len(evicted) >= 1 and len(done) >= 1            # the pool (30 blocks of 4 tokens) is too small for 12 full traces
        assert o.pool.used == 0 and o.pool.status == 0           # all KV returned, nobody ever failed to get a block
        o.pool.check_invariants()
        assert all(len(e["evicted"]) <= 4 for e in log)
        # the vote: recompute by brute force from the recorded final scores
        tot = {}
        for t in done:
            s, a = o.finished[t]
            tot[a] = tot.get(a, 0.0) + s
        best = max(tot.values())
        assert ans == min(a for a, w in tot.items() if w == best)


def test_evicted_trace_is_the_argmin_of_the_running_means():
    o, toks, hid, answers = _random_run(5, max_evictions=1)
    for i in range(len(toks)):
        if not o.live():
            break
        # scores the eviction will see: means after this iteration's scoring; recompute them independently
        sums, cnts = o.ts.sum.copy(), o.ts.cnt.copy()
        live = o.live()
        ev = o.iteration(toks[i], hid[i], answers)
        for t in live:
            if ev["mask"][t]:
                sums[t] += ev["step_scores"][t]; cnts[t] += 1
        if ev["evicted"]:
            cand = [t for t in live if t not in ev["finished"]]
            mean = {t: (sums[t] / cnts[t] if cnts[t] else 1.0) for t in cand}
            worst = min(cand, key=lambda t: (mean[t], -t))       # lowest mean; among equals the larger id goes
            assert ev["evicted"] == [worst]
