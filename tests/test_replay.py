"""The preempt-and-recompute schedule driven against the oracle pool: every trace completes, all KV returns, and the
waiting the schedule produces disappears when the pool is large enough."""
import numpy as np

from oracle.kv_pool import KVPoolOracle
from paper_2601_09093_b200.replay import preempt_and_recompute


class OracleOps:
    def __init__(self, pool):
        self.p = pool
        self.log = []

    def free(self):
        return self.p.free_count

    def fork_all(self, n, prompt_len):
        ids = self.p.fork_prefix(n, prompt_len)
        assert len(ids) == n
        return ids

    def fork_one(self, seq_len):
        ids = self.p.fork_prefix(1, seq_len)
        assert len(ids) == 1, "the schedule admitted a trace that does not fit"
        return ids[0]

    def append(self, ids):
        assert all(self.p.append_kv(ids, 1)), "the schedule let an append fail"

    def release(self, ids):
        for t in ids:
            self.p.release_trace(t)

    finish = release


def _run(num_blocks, n=12, prompt=32, lo=60, hi=200, seed=3):
    g = np.random.default_rng(seed)
    final = [int(x) for x in g.integers(lo, hi, size=n)]
    pool = KVPoolOracle(1, 1, 8, 16, num_blocks, 400, -(-hi // 16) + 1, store_payload=False)
    c = preempt_and_recompute(OracleOps(pool), final, prompt, 16)
    assert c["unfinished"] == 0 and pool.status == 0
    assert pool.free_count == num_blocks and not pool.live.any()          # every block came back
    pool.check_invariants()
    assert c["decode_steps"] == sum(final) - n * prompt + 0 * c["preemptions"]
    return c, final


def test_large_pool_never_waits():
    c, final = _run(num_blocks=400)
    assert c["preemptions"] == 0 and c["waiting_trace_iterations"] == 0 and c["recomputed_tokens"] == 0
    assert c["iterations"] == max(final) - 32


def test_small_pool_preempts_waits_and_recomputes():
    c, final = _run(num_blocks=24)
    assert c["preemptions"] > 0 and c["waiting_trace_iterations"] > 0 and c["recomputed_tokens"] > 0
    assert c["iterations"] > max(final) - 32                              # the queue stretches the run
    c2, _ = _run(num_blocks=32)
    assert c2["waiting_trace_iterations"] < c["waiting_trace_iterations"]
