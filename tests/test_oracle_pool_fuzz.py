"""Random operation sequences on the oracle pool alone: its invariants hold after every operation, blocks are
conserved, and an independent recount of the reference counts from the block tables agrees."""
import numpy as np
import pytest

from oracle.kv_pool import KVPoolOracle


def _recount(o):
    """Reference counts recomputed from scratch: how many live traces map each block."""
    rc = np.zeros(o.num_blocks, dtype=np.int64)
    for t in range(o.max_traces):
        if o.live[t]:
            pages = -(-int(o.seq_lens[t]) // o.P)
            for b in o.block_table[t, :pages]:
                rc[int(b)] += 1
            assert (o.block_table[t, pages:] == -1).all()
        else:
            assert o.seq_lens[t] == 0 and (o.block_table[t] == -1).all()
    return rc


@pytest.mark.parametrize("seed", range(25))
def test_invariants_under_random_operations(seed):
    g = np.random.default_rng(5000 + seed)
    nb, T, max_pages, P = int(g.integers(20, 90)), 20, int(g.integers(4, 12)), 16
    o = KVPoolOracle(1, 1, 4, P, nb, T, max_pages, store_payload=False)
    for step in range(120):
        live = [t for t in range(T) if o.live[t]]
        op = g.choice(["fork", "append", "append", "prune", "release"])
        if op == "fork" or not live:
            o.fork_prefix(int(g.integers(1, 4)), int(g.choice([0, 3, 16, 33, 64])))      # may fail: flagged, no effect
        elif op == "append":
            ids = [int(x) for x in g.choice(live, size=int(g.integers(1, len(live) + 1)), replace=False)]
            before = o.free_count
            ok = o.append_kv(ids, int(g.choice([1, 1, 5, 16, 40])))
            assert len(ok) == len(ids) and o.free_count <= before
        elif op == "prune":
            scores = g.random(T).astype(np.float32)
            thr, kf = float(g.choice([0.2, 0.7, 1.0])), float(g.choice([-1.0, 0.5, 1.0]))
            fired = o.saturated(thr)
            n_live = len(live)
            ev = o.prune_if_saturated(scores, thr, kf)
            if not fired:
                assert ev == []
            else:
                assert len(ev) == n_live - o.n_keep(kf, n_live)
                kept = [t for t in live if t not in ev]
                # every kept trace ranks at least as high as every evicted one (score descending, id ascending)
                assert all((scores[k], -k) >= (scores[e], -e) for k in kept for e in ev)
        else:
            o.release_trace(int(g.choice(live)))
        o.status = 0
        o.check_invariants()
        rc = _recount(o)
        assert (rc == o.refcount).all()
        assert o.free_count == nb - int((rc > 0).sum())
        assert sorted(o.free_list) == sorted(np.flatnonzero(rc == 0).tolist())
