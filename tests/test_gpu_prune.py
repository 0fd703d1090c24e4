"""GPU parity of prune_if_saturated / release against the oracle's rule: bit-exact sets and free list."""
import os

import numpy as np
import pytest
import torch

from oracle import scorer as OS
from paper_2601_09093_b200 import binding as B
from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W

from gpu_common import Twin

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _lines(name):
    with open(os.path.join(GOLD, name)) as f:
        return [l.strip() for l in f if l.strip() and not l.startswith("#")]


def _prune_both(tw, scores, threshold, keep_frac):
    sc = torch.from_numpy(np.asarray(scores, dtype=np.float32)).cuda()
    ids, n = tw.gpu.prune_if_saturated(sc, threshold, keep_frac)
    n = int(n.item())
    got = ids[:n].cpu().tolist()
    want = tw.ora.prune_if_saturated(np.asarray(scores, dtype=np.float32), threshold, keep_frac)
    assert got == want, (got, want)
    tw.assert_meta_equal()
    return got


@pytest.mark.parametrize("line", _lines("prune_hand_examples.txt"))
def test_hand_examples(line):
    scores, kf, kept, evicted = [x.split() for x in line.split("|")]
    scores = [float(x) for x in scores]
    n = len(scores)
    cfg = W.scaled(W.C0, prefix_len=16)
    tw = Twin(cfg, n * 3 + 2, 5, n, store_payload=False)
    ids, _ = tw.fork(n, 16)
    tw.append(ids, 32)
    got = _prune_both(tw, scores, 0.5, float(kf[0]))
    assert got == [int(x) for x in evicted]
    assert tw.status() == (0, 0)


def test_not_saturated_is_a_noop():
    cfg = W.scaled(W.C0, prefix_len=16)
    tw = Twin(cfg, 100, 5, 4, store_payload=False)
    ids, _ = tw.fork(4, 16)
    tw.append(ids, 32)
    assert _prune_both(tw, [0.1, 0.2, 0.3, 0.4], 0.95, 0.5) == []


def test_trigger_boundary_matches_integer_predicate():
    cfg = W.scaled(W.C0, prefix_len=4, page_size=4, head_dim=64)
    tw = Twin(cfg, 10, 8, 2, store_payload=False)
    ids, _ = tw.fork(2, 4)
    tw.append(ids, 8)                                  # used 5, both on a page boundary: need 2
    for thr, fires in ((0.75, False), (0.7, True), (0.6, True)):
        assert tw.ora.saturated(thr) is fires
    assert _prune_both(tw, [0.5, 0.4], 0.75, 0.5) == []
    assert _prune_both(tw, [0.5, 0.4], 0.7, 0.5) == [1]


def test_shared_prefix_blocks_return_only_with_the_last_sharer():
    cfg = W.scaled(W.C0, prefix_len=40)                # 2 shared pages + a private partial page each
    tw = Twin(cfg, 64, 8, 6, store_payload=False)
    ids, _ = tw.fork(6, 40)
    tw.append(ids, 30)
    _prune_both(tw, [0.9, 0.1, 0.8, 0.2, 0.7, 0.3], 0.01, 0.5)
    _prune_both(tw, [0.9, 0.1, 0.8, 0.2, 0.7, 0.3], 0.01, -1.0)
    _prune_both(tw, [0.9, 0.1, 0.8, 0.2, 0.7, 0.3], 0.01, -1.0)
    _prune_both(tw, [0.9, 0.1, 0.8, 0.2, 0.7, 0.3], 0.01, 0.5)      # keep_frac of one trace keeps it
    st = tw.gpu.stats()
    assert st["live_traces"] == 1
    tw.gpu.release_traces(torch.tensor([0], dtype=torch.int32, device="cuda"))
    tw.ora.release_trace(0)
    tw.assert_meta_equal()
    assert tw.gpu.stats()["used"] == 0


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_random_pools_with_ties_and_nans(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(3, 130))
    cfg = W.scaled(W.C0, prefix_len=int(rng.integers(0, 50)))
    lens = rng.integers(0, 2500, size=n)
    tw = Twin(cfg, int(sum(-(-(cfg.prefix_len + l) // 16) for l in lens)) + 40, 170, n, shuffle=bool(seed % 2),
              store_payload=False)
    ids, _ = tw.fork(n, cfg.prefix_len)
    for sel, inc in H.ragged_append_plan(lens):
        tw.append([ids[i] for i in sel], inc)
    scores = rng.choice([0.1, 0.25, 0.5, 0.75, np.nan], size=n).astype(np.float32)
    for kf in (0.5, -1.0, 0.3, 0.5):
        _prune_both(tw, scores, 0.2, kf)
    assert tw.status() == (0, 0)


def test_release_of_finished_traces_and_bad_ids():
    cfg = W.scaled(W.C0, prefix_len=16)
    tw = Twin(cfg, 40, 6, 5, store_payload=False)
    ids, _ = tw.fork(5, 16)
    tw.append(ids, 40)
    tw.gpu.release_traces(torch.tensor([3, 1, 9], dtype=torch.int32, device="cuda"))
    tw.ora.release_trace(3); tw.ora.release_trace(1)
    tw.assert_meta_equal()
    assert tw.gpu.last_error()[1] == 1 << 3


def test_memory_saturated_cycles_scaled_down():
    """The structure of the memory-saturated benchmark at 1/256 of its pool: 64 traces grow one
    token per step from a shared prompt; scores come from score_steps on seeded hidden states;
    at 95 % the top half survives; 5 cycles.  Metadata must track the oracle bit for bit, and a
    prune that fired must leave room for every survivor's next token (no waiting queue)."""
    cfg = W.scaled(W.C3, num_layers=1, num_kv_heads=1, num_q_heads=4, head_dim=64, prefix_len=32,
                   scorer_D=256, scorer_m=64, dtype="fp32")
    T, nb = 64, 256
    tw = Twin(cfg, nb, nb, T, store_payload=False)
    ids, _ = tw.fork(T, cfg.prefix_len)
    (W1b, W1x), (b1b, b1x), (w2b, w2x), b2 = W.scorer_weights(cfg, std=0.2)
    wts = B.ScorerWeights(H.to_device(W1b, "fp32"), H.to_device(b1b, "fp32"), H.to_device(w2b, "fp32"), b2, B.STEP_FP32)
    ts = OS.TraceScores(T)
    live = list(ids)
    cycles, step = 0, 0
    while cycles < 5 and step < 5000:
        step += 1
        tw.append(live, 1)
        hb, hx = W.normal(cfg.seed, W.TID_HID, (T, cfg.scorer_D), "fp32", sub=step)
        mask = W.boundary_mask(cfg, T, sub=step, density=1.0 / 4)
        mask[[t for t in range(T) if t not in live]] = 0
        g = tw.gpu.score_steps(H.to_device(hb, "fp32"), torch.from_numpy(mask).cuda(), None, wts).cpu().numpy()
        ts.update(g, mask)
        scores = tw.gpu.views()["trace_scores"].cpu().numpy()
        np.testing.assert_allclose(scores[live], ts.scores()[live], atol=1e-6)
        pid, n = tw.gpu.prune_if_saturated(None, 0.95, 0.5)          # the pool's own running means
        n = int(n.item())
        got = pid[:n].cpu().tolist()
        want = tw.ora.prune_if_saturated(scores, 0.95, 0.5, on_evict=ts.clear)
        assert got == want
        if got:
            cycles += 1
            live = [t for t in live if t not in got]
            assert len(live) == 64 >> cycles
        tw.assert_meta_equal()
        assert tw.status() == (0, 0), "a survivor could not be scheduled"
    assert cycles == 5 and len(live) == 2
