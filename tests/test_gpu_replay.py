"""The preempt-and-recompute schedule (what an engine without pruning does when the KV pool fills: Sec. 2 "Latency
Bottleneck", Table 3's waiting) driving a CUDA pool and the oracle's pool in lockstep: every pool operation the
schedule issues goes to both, and the metadata must agree bit for bit after every preemption, after every
reconstruction, and at the end."""
import numpy as np
import pytest
import torch

from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W
from paper_2601_09093_b200.replay import preempt_and_recompute

from gpu_common import Twin

pytestmark = pytest.mark.gpu


class LockstepOps:
    """The five operations of the schedule on a Twin (CUDA pool + oracle pool, bookkeeping only)."""

    def __init__(self, tw, prompt_max):
        self.tw, self.checks = tw, 0
        c = tw.cfg
        self.kbuf = torch.zeros((c.num_layers, c.num_kv_heads, prompt_max, c.head_dim), dtype=tw.gpu.torch_dtype, device="cuda")
        self.knew = torch.zeros((tw.gpu.max_traces, 1, c.num_layers, c.num_kv_heads, c.head_dim), dtype=tw.gpu.torch_dtype, device="cuda")

    def _dev(self, ids):
        return torch.tensor(list(ids), dtype=torch.int32, device="cuda")

    def free(self):
        f = self.tw.gpu.stats()["free"]
        assert f == self.tw.ora.free_count
        return f

    def fork_all(self, n, S):
        ids = self.tw.gpu.fork_prefix(n, S, self.kbuf[:, :, :S].contiguous(), self.kbuf[:, :, :S].contiguous())
        oids = self.tw.ora.fork_prefix(n, S)
        assert ids == oids and len(ids) == n
        return ids

    def fork_one(self, S):
        t = self.fork_all(1, S)[0]
        self.tw.assert_meta_equal(); self.checks += 1          # after every reconstruction
        return t

    def append(self, ids):
        self.tw.gpu.append_kv(self._dev(ids), 1, self.knew[:len(ids)], self.knew[:len(ids)])
        assert all(self.tw.ora.append_kv(list(ids), 1))

    def release(self, ids):
        self.tw.gpu.release_traces(self._dev(ids))
        for t in ids:
            self.tw.ora.release_trace(t)
        self.tw.assert_meta_equal(); self.checks += 1          # after every preemption

    def finish(self, ids):
        self.tw.gpu.finish_traces(self._dev(ids), None)
        for t in ids:
            self.tw.ora.release_trace(t)


@pytest.mark.parametrize("num_blocks,shuffle", [(40, False), (56, True)])
def test_preempt_and_recompute_in_lockstep_with_the_oracle_pool(num_blocks, shuffle):
    g = np.random.default_rng(5 + num_blocks)
    n, prompt, P = 12, 40, 16                                  # a prompt with a partial last page: private copies
    final = [int(x) for x in g.integers(90, 260, size=n)]
    cfg = W.scaled(W.C1, n_traces=n, num_layers=1, num_q_heads=8, num_kv_heads=2, prefix_len=prompt, seed=99)
    tw = Twin(cfg, num_blocks, -(-max(final) // P) + 1, 400, shuffle=shuffle, store_payload=False)
    ops = LockstepOps(tw, max(final))
    c = preempt_and_recompute(ops, final, prompt, P)
    assert c["unfinished"] == 0 and c["preemptions"] > 0 and c["recomputed_tokens"] > 0
    assert ops.checks >= 2 * c["preemptions"]
    tw.assert_meta_equal()
    st = tw.gpu.stats()
    assert st["used"] == 0 and st["live_traces"] == 0          # every block came back
    assert tw.status() == (0, 0)
