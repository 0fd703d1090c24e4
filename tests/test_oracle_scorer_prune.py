"""Pins for oracle/scorer.py and oracle/kv_pool.py."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import scorer as S
from oracle.kv_pool import KVPoolOracle, weighted_vote, ERR_NO_BLOCKS, ERR_BAD_TRACE, ERR_CAPACITY

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _lines(name):
    with open(os.path.join(GOLD, name)) as f:
        return [l.strip() for l in f if l.strip() and not l.startswith("#")]


# ------------------------------------------------------------------ scorer
def test_hand_worked_example():
    want = float(_lines("scorer_hand_example.txt")[0].split()[1])
    y = S.step_score([1, 2], [[1, -1], [0.5, 2]], [0, -1], [2, -1], 0.5)
    assert abs(y - want) < 1e-15
    assert abs(want - 1.0 / (1.0 + 20.085536923187668)) < 1e-15


def test_flops_match_paper_formula():
    for line in _lines("scorer_flops.txt"):
        m, d, flops = (int(x) for x in line.split())
        assert S.scorer_flops(m, d) == flops == 2 * m * (d + 1)


def test_special_cases():
    rng = np.random.default_rng(0)
    h, W1, b1, w2 = rng.standard_normal(8), rng.standard_normal((5, 8)), rng.standard_normal(5), rng.standard_normal(5)
    assert S.step_score(h, W1, b1, np.zeros(5), 0.0) == 0.5                    # zero w2, b2 = 0
    assert abs(S.step_score(h, W1, b1, np.zeros(5), 1.0) - 1 / (1 + math.exp(-1))) < 1e-15
    # zero W1: y = sigmoid(w2 . ReLU(b1) + b2)
    z = sum(w * max(b, 0.0) for w, b in zip(w2, b1)) + 0.25
    assert abs(S.step_score(h, np.zeros((5, 8)), b1, w2, 0.25) - 1 / (1 + math.exp(-z))) < 1e-14
    # all pre-activations negative: ReLU kills them, only b2 is left
    assert S.step_score(np.ones(8), -np.ones((5, 8)), np.zeros(5), w2, 0.0) == 0.5
    # monotone in b2
    ys = [S.step_score(h, W1, b1, w2, b) for b in (-2, -1, 0, 1, 2)]
    assert all(a < b for a, b in zip(ys, ys[1:]))


def test_matches_torch_mlp():
    rng = np.random.default_rng(1)
    D, m, M = 96, 40, 7
    H, W1, b1, w2, b2 = rng.standard_normal((M, D)), rng.standard_normal((m, D)) * .1, rng.standard_normal(m) * .1, rng.standard_normal(m) * .3, 0.2
    net = torch.nn.Sequential(torch.nn.Linear(D, m), torch.nn.ReLU(), torch.nn.Linear(m, 1), torch.nn.Sigmoid()).double()
    with torch.no_grad():
        net[0].weight.copy_(torch.from_numpy(W1)); net[0].bias.copy_(torch.from_numpy(b1))
        net[2].weight.copy_(torch.from_numpy(w2)[None]); net[2].bias.fill_(b2)
        want = net(torch.from_numpy(H))[:, 0].numpy()
    mask = np.array([1, 0, 1, 1, 0, 1, 1])
    got = S.score_steps(H, mask, W1, b1, w2, b2)
    np.testing.assert_allclose(got[mask == 1], want[mask == 1], atol=1e-14)
    assert np.isnan(got[mask == 0]).all()


def test_running_mean_golden():
    ts = S.TraceScores(2, unscored_score=1.0)
    assert ts.score(0) == 1.0
    for line in _lines("running_mean.txt"):
        y, mean = (float(x) for x in line.split())
        ts.update([y, 0.99], [1, 0])                      # row 1 is not a boundary: ignored
        assert abs(ts.score(0) - mean) < 1e-15
    assert ts.cnt[1] == 0 and ts.score(1) == 1.0


def test_running_mean_row_trace_and_order():
    ts = S.TraceScores(3)
    ts.update([0.1, 0.5, 0.9, 0.3], [1, 1, 1, 1], row_trace=[2, 0, 2, 0])
    assert abs(ts.score(2) - 0.5) < 1e-15 and abs(ts.score(0) - 0.4) < 1e-15 and ts.cnt[1] == 0


# ------------------------------------------------------------------- prune
def _pool_with_scores(n, blocks_each, num_blocks=None, P=4):
    num_blocks = num_blocks or n * blocks_each + 2
    pool = KVPoolOracle(1, 1, 2, P, num_blocks, n, blocks_each + 2, store_payload=False)
    ids = pool.fork_prefix(n, P)                           # one shared page
    pool.append_kv(ids, (blocks_each - 1) * P)
    return pool


@pytest.mark.parametrize("line", _lines("prune_hand_examples.txt"))
def test_prune_hand_examples(line):
    scores, kf, kept, evicted = [x.split() for x in line.split("|")]
    scores = np.array([float(x) for x in scores], dtype=np.float32)
    n = len(scores)
    pool = _pool_with_scores(n, 3)
    got = pool.prune_if_saturated(scores, threshold=0.5, keep_frac=float(kf[0]))
    assert got == [int(x) for x in evicted]
    assert [t for t in range(n) if pool.live[t]] == [int(x) for x in kept]
    pool.check_invariants()


def test_not_saturated_is_a_noop():
    pool = _pool_with_scores(4, 3, num_blocks=100)
    before = (list(pool.free_list), pool.block_table.copy(), pool.live.copy())
    assert pool.prune_if_saturated(np.zeros(4, np.float32), threshold=0.95, keep_frac=0.5) == []
    assert before[0] == pool.free_list and np.array_equal(before[1], pool.block_table) and np.array_equal(before[2], pool.live)


def test_trigger_predicate_by_hand():
    # total 10 blocks, P = 4.  2 traces, shared 1 page, then 2 private pages each: used = 5.
    pool = KVPoolOracle(1, 1, 2, 4, 10, 2, 8, store_payload=False)
    ids = pool.fork_prefix(2, 4); pool.append_kv(ids, 8)
    assert pool.used == 5 and list(pool.seq_lens[:2]) == [12, 12]
    # both traces sit on a page boundary: the next step needs 2 blocks -> used + need = 7
    assert pool.saturated(0.6) is True          # limit = floor(6.0000002) = 6 ; 7 > 6
    assert pool.saturated(0.75) is False        # limit 7 ; 7 > 7 false
    pool.append_kv(ids, 1)                       # now mid-page: need = 0, used = 7
    assert pool.saturated(0.6) is True and pool.saturated(0.75) is False
    # threshold 1.0 = the paper's sentence: full means the next step cannot be scheduled
    pool.append_kv(ids, 3); pool.append_kv(ids[:1], 4)   # used = 8, trace 0 at 20, trace 1 at 16
    assert pool.used == 8 and pool.saturated(1.0) is False    # need 2, 8 + 2 = 10 fits exactly
    pool.append_kv(ids[:1], 1)                   # used 9, need: trace 1 on boundary -> 1; 10 <= 10
    assert pool.saturated(1.0) is False
    pool.append_kv(ids[1:], 1)                   # used 10, need 0
    assert pool.saturated(1.0) is False
    pool.append_kv(ids, 3)                       # trace 0 at 24 (boundary), used 10 -> 10 + 1 > 10
    assert pool.saturated(1.0) is True


def test_float32_threshold_rounding_is_part_of_the_rule():
    pool = KVPoolOracle(1, 1, 2, 4, 10, 2, 8, store_payload=False)
    ids = pool.fork_prefix(2, 4); pool.append_kv(ids, 8)      # used 5, need 2 -> 7
    # float32(0.7) = 0.699999988..., times 10 -> 6.99999988 -> limit 6 -> saturated
    assert math.floor(float(np.float32(0.7)) * 10) == 6
    assert pool.saturated(0.7) is True


def test_reclaim_order_refcounts_and_shared_prefix():
    P = 4
    pool = KVPoolOracle(1, 1, 2, P, 20, 4, 6, store_payload=False)
    ids = pool.fork_prefix(4, 2 * P)                     # shared blocks 0, 1 (first pops)
    assert list(pool.block_table[0, :2]) == [0, 1] and pool.refcount[0] == 4
    pool.append_kv(ids, P)                               # private: t0->2, t1->3, t2->4, t3->5
    assert [int(pool.block_table[t, 2]) for t in range(4)] == [2, 3, 4, 5]
    fl0 = list(pool.free_list)
    ev = pool.prune_if_saturated(np.array([0.9, 0.1, 0.8, 0.2], np.float32), threshold=0.1, keep_frac=0.5)
    assert ev == [1, 3]
    # shared pages stay (two sharers left); private pages return in (trace, page) order
    assert pool.free_list == fl0 + [3, 5]
    assert pool.refcount[0] == 2 and pool.refcount[1] == 2
    pool.check_invariants()
    ev = pool.prune_if_saturated(np.array([0.9, 0.0, 0.8, 0.0], np.float32), threshold=0.1, keep_frac=-1.0)
    assert ev == [2] and pool.free_list == fl0 + [3, 5, 4]
    # evicting the last sharer returns the shared pages too, in page order, before its private page
    pool.release_trace(0)
    assert pool.free_list == fl0 + [3, 5, 4, 0, 1, 2]
    pool.check_invariants()
    assert pool.used == 0


def test_fork_with_partial_last_page_gives_private_tail_blocks():
    P = 4
    pool = KVPoolOracle(1, 1, 2, P, 20, 3, 6, store_payload=False)
    ids = pool.fork_prefix(3, 6)                          # 1 full shared page + 2 tokens
    assert ids == [0, 1, 2]
    assert [int(pool.block_table[t, 0]) for t in ids] == [0, 0, 0]
    assert [int(pool.block_table[t, 1]) for t in ids] == [1, 2, 3]
    assert pool.refcount[0] == 3 and all(pool.refcount[b] == 1 for b in (1, 2, 3))
    pool.check_invariants()


def test_append_n_times_one_equals_append_n():
    rng = np.random.default_rng(5)
    def build(bulk):
        pool = KVPoolOracle(2, 2, 4, 4, 64, 3, 10, store_payload=True)
        kp, vp = rng0.standard_normal((2, 2, 5, 4)), rng0.standard_normal((2, 2, 5, 4))
        ids = pool.fork_prefix(3, 5, kp, vp)
        kn, vn = rng0.standard_normal((3, 9, 2, 2, 4)), rng0.standard_normal((3, 9, 2, 2, 4))
        if bulk:
            pool.append_kv(ids, 9, kn, vn)
        else:
            for j in range(9):
                pool.append_kv(ids, 1, kn[:, j:j + 1], vn[:, j:j + 1])
        return pool
    rng0 = np.random.default_rng(5); a = build(True)
    rng0 = np.random.default_rng(5); b = build(False)
    assert np.array_equal(a.seq_lens, b.seq_lens)
    # block placement differs (page-by-page vs trace-by-trace) but logical content must not
    from oracle.attention import gather_trace_kv
    for t in range(3):
        for l in range(2):
            Ka, Va = gather_trace_kv(a.k_pages[l], a.v_pages[l], a.block_table[t], 14)
            Kb, Vb = gather_trace_kv(b.k_pages[l], b.v_pages[l], b.block_table[t], 14)
            assert np.array_equal(Ka, Kb) and np.array_equal(Va, Vb)
    a.check_invariants(); b.check_invariants()


def test_error_conditions_set_status_and_skip():
    pool = KVPoolOracle(1, 1, 2, 4, 3, 2, 2, store_payload=False)
    ids = pool.fork_prefix(2, 4)                          # 1 shared block, 2 free
    assert pool.append_kv([0, 1, 5], 4) == [True, True, False] and pool.status == 1 << ERR_BAD_TRACE
    pool.status = 0
    assert pool.append_kv([0], 1) == [False] and pool.status == 1 << ERR_CAPACITY   # third page > max_pages
    pool2 = KVPoolOracle(1, 1, 2, 4, 2, 2, 4, store_payload=False)
    pool2.fork_prefix(2, 4)
    assert pool2.append_kv([0, 1], 4) == [True, False] and pool2.status == 1 << ERR_NO_BLOCKS
    pool2.check_invariants()


def test_after_a_prune_that_fired_survivors_can_append():
    # the paper's claim that memory-triggered pruning leaves nobody waiting (Table 3: wait = 0)
    P = 4
    pool = KVPoolOracle(1, 1, 2, P, 40, 8, 64, store_payload=False)
    ids = pool.fork_prefix(8, P)
    scores = np.linspace(0.1, 0.9, 8).astype(np.float32)
    live = list(ids)
    fired = 0
    for step in range(150):
        ev = pool.prune_if_saturated(scores, threshold=1.0, keep_frac=-1.0)
        fired += len(ev)
        live = [t for t in live if t not in ev]
        ok = pool.append_kv(live, 1)
        if pool.status:
            # only acceptable once a single trace is left and even it does not fit
            assert len(live) == 1 and pool.status == 1 << ERR_NO_BLOCKS
            break
        assert all(ok)
        pool.check_invariants()
    assert fired == 7 and live == [7]                       # worst scores go first, one at a time


def test_bytes_per_token_of_the_8b_layout():
    pool = KVPoolOracle(36, 8, 128, 16, 4, 1, 1, store_payload=False)
    assert pool.bytes_per_token(2) == 147456


def test_weighted_vote():
    assert weighted_vote([7, 3, 7, 3, 5], [0.2, 0.5, 0.2, 0.1, 0.55]) == 3      # 0.6 vs 0.4 vs 0.55
    assert weighted_vote([1, 2], [0.5, 0.5]) == 1
    assert weighted_vote([], []) is None
