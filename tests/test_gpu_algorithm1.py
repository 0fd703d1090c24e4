"""GPU parity of the Algorithm 1 driver (iteration, completion, vote, whole run) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import attention as OA
from oracle.algorithm1 import Algorithm1Oracle
from oracle.kv_pool import KVPoolOracle, weighted_vote
from paper_2601_09093_b200 import binding as B
from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W

from test_oracle_algorithm1 import VOCAB, load_hand_example

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _meta_equal(pool, ora):
    v = pool.views()
    torch.cuda.synchronize()
    fc = int(v["free_count"].item())
    assert v["free_list"][:fc].cpu().tolist() == ora.free_list
    np.testing.assert_array_equal(v["seq_lens"].cpu().numpy(), ora.seq_lens)
    np.testing.assert_array_equal(v["live"].cpu().numpy().astype(bool), ora.live)
    np.testing.assert_array_equal(v["refcount"].cpu().numpy(), ora.refcount)
    np.testing.assert_array_equal(v["block_table"].cpu().numpy(), ora.block_table)
    ora.check_invariants()


def test_hand_worked_example_on_the_gpu():
    rows, answers, vote = load_hand_example()
    cfg = W.scaled(W.C0, num_layers=1, num_q_heads=1, num_kv_heads=1, head_dim=4, page_size=2, scorer_D=1, scorer_m=1)
    pool = H.make_pool(cfg, 6, 8, 3)
    z = torch.zeros((1, 1, 2, 4), dtype=torch.float32, device=DEV)
    assert pool.fork_prefix(3, 2, z, z) == [0, 1, 2]
    one = torch.ones((1, 1), dtype=torch.float32, device=DEV)
    wts = B.ScorerWeights(one, torch.zeros(1, device=DEV), torch.ones(1, device=DEV), 0.0, B.STEP_FP32)
    table = B.step_end_table_from_vocab(VOCAB).to(DEV)
    ans = torch.tensor(answers, dtype=torch.int32, device=DEV)
    kv = torch.zeros((3, 1, 1, 1, 4), dtype=torch.float32, device=DEV)
    ts_out = torch.empty(3, dtype=torch.float32, device=DEV)
    done, gone = set(), set()
    for r in rows:
        tok = torch.tensor(r["tokens"], dtype=torch.int32, device=DEV)
        hid = torch.tensor(r["h"], dtype=torch.float32, device=DEV).reshape(3, 1)
        pool.algorithm1_iteration(tok, 2, table, ans, None, kv, kv, hid, wts, 1.0, -1.0, trace_scores_out=ts_out)
        v, vv = pool.views(), pool.vote_views()
        live = v["live"].cpu().numpy().astype(bool)
        fin = vv["finished"].cpu().numpy().astype(bool)
        new_done = {t for t in range(3) if fin[t]} - done
        new_gone = {t for t in range(3) if not live[t] and not fin[t]} - gone
        assert sorted(new_done) == r["finished"] and sorted(new_gone) == r["evicted"]
        done |= new_done; gone |= new_gone
        assert pool.stats()["used"] == r["used"]
        got = ts_out.cpu().numpy()
        for t, want in enumerate(r["scores"]):
            if want is not None:
                assert abs(got[t] - want) < 1e-6
    a, w, n = pool.weighted_vote()
    assert int(a.item()) == vote and abs(float(w.item()) - 0.75) < 1e-6 and int(n.item()) == 2
    assert pool.last_error() == (0, 0)


def test_finish_traces_and_vote_ties_and_missing_answers():
    cfg = W.scaled(W.C0, prefix_len=16)
    pool = H.make_pool(cfg, 40, 6, 6)
    ora = KVPoolOracle(1, 1, 64, 16, 40, 6, 6, store_payload=False)
    z = torch.zeros((1, 1, 16, 64), dtype=torch.float32, device=DEV)
    ids = pool.fork_prefix(6, 16, z, z); ora.fork_prefix(6, 16)
    kv = torch.zeros((6, 20, 1, 1, 64), dtype=torch.float32, device=DEV)
    pool.append_kv(torch.arange(6, dtype=torch.int32, device=DEV), 20, kv, kv); ora.append_kv(ids, 20)
    # scores 0.5 each (exactly representable): answers 9, 4, 9, 4 tie at 1.0 -> the smaller id wins; trace 4 has no answer
    pool.views()["trace_scores"][:6] = 0.5
    a0, _, n0 = pool.weighted_vote()
    assert int(a0.item()) == -1 and int(n0.item()) == 0
    fin = torch.tensor([3, 0, 2, 1, 4, 17], dtype=torch.int32, device=DEV)
    ans = torch.tensor([4, 9, 9, 4, -1, 1], dtype=torch.int32, device=DEV)
    pool.finish_traces(fin, ans)
    for t in (3, 0, 2, 1, 4):
        ora.release_trace(t)
    _meta_equal(pool, ora)
    assert pool.last_error()[1] == 1 << 3                          # id 17 names no trace
    a, w, n = pool.weighted_vote()
    assert (int(a.item()), float(w.item()), int(n.item())) == (4, 1.0, 5)
    assert weighted_vote([4, 9, 9, 4], [0.5] * 4) == 4


def _driver_case(seed, n, iters, num_blocks, with_attention, p_eos=0.02):
    cfg = W.scaled(W.C1, n_traces=n, num_layers=2, num_q_heads=8, num_kv_heads=2, prefix_len=32, scorer_D=256,
                   scorer_m=64, seed=seed)
    vocab = W.synthetic_vocab(seed, 500, step_end_frac=0.1)
    eos = 0
    table = B.step_end_table_from_vocab(vocab)
    ends = np.flatnonzero(table.numpy())
    toks = np.stack([W.token_ids(seed, n, len(vocab), ends, 0.25, sub=i) for i in range(iters)])
    toks[toks == eos] = 1
    toks[W.rng(seed, W.TID_TOK, 999).random(toks.shape) < p_eos] = eos
    toks[iters - 1] = eos
    answers = W.rng(seed, W.TID_ANS).integers(0, 5, size=n).astype(np.int32)
    (W1b, W1x), (b1b, b1x), (w2b, w2x), b2 = W.scorer_weights(cfg, std=0.3, bias_std=0.05)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16"), H.to_device(b1b, "bf16"), H.to_device(w2b, "bf16"), b2, B.STEP_BF16)
    pool = H.make_pool(cfg, num_blocks, 64, n)
    ora_pool = KVPoolOracle(2, 2, 128, 16, num_blocks, n, 64, store_payload=with_attention)
    shp = (2, 2, 32, 128)
    kb, kx = W.normal(seed, W.TID_KPRE, shp, "bf16"); vb, vx = W.normal(seed, W.TID_VPRE, shp, "bf16")
    pool.fork_prefix(n, 32, H.to_device(kb, "bf16"), H.to_device(vb, "bf16"))
    ora_pool.fork_prefix(n, 32, kx, vx)
    return cfg, vocab, eos, table.to(DEV), toks, answers, (W1x, b1x, w2x, b2), wts, pool, ora_pool


@pytest.mark.parametrize("seed,keep_frac,max_ev", [(11, -1.0, 2), (12, 0.5, 1)])
def test_iteration_by_iteration_against_the_oracle(seed, keep_frac, max_ev):
    n, iters = 16, 160
    cfg, vocab, eos, table, toks, answers, wx, wts, pool, ora_pool = _driver_case(seed, n, iters, 26, True)
    ora = Algorithm1Oracle(ora_pool, n, *wx, vocab, eos, 1.0, keep_frac, max_evictions=max_ev)
    ans_dev = torch.from_numpy(answers).to(DEV)
    ts_out = torch.empty(n, dtype=torch.float32, device=DEV)
    mask_out = torch.empty(n, dtype=torch.uint8, device=DEV)
    n_ev = n_fin = 0
    for i in range(iters):
        if not ora.live():
            break
        shp = (n, 1, 2, 2, 128)
        kb, kx = W.normal(seed, W.TID_KNEW, shp, "bf16", sub=i); vb, vx = W.normal(seed, W.TID_VNEW, shp, "bf16", sub=i)
        hb, hx = W.normal(seed, W.TID_HID, (n, cfg.scorer_D), "bf16", sub=i)
        qb, qx = W.normal(seed, W.TID_Q, (2, n, 8, 128), "bf16", sub=i)
        live_before = ora.live()
        att, ys = pool.algorithm1_iteration(torch.from_numpy(toks[i]).to(DEV), eos, table, ans_dev, H.to_device(qb, "bf16"),
                                            H.to_device(kb, "bf16"), H.to_device(vb, "bf16"), H.to_device(hb, "bf16"), wts,
                                            1.0, keep_frac, max_evictions=max_ev, trace_scores_out=ts_out,
                                            boundary_mask_out=mask_out)
        g_scores = ts_out.cpu().numpy()
        g_ys = ys.cpu().numpy()
        # both sides take the eviction decision on the device's float32 scores
        ev = ora.iteration(toks[i], hx, answers, kx, vx, rank_scores=g_scores, step_scores=g_ys,
                           q=qx if i % 16 == 0 else None)
        if ev["attention"] is not None:
            err = np.abs(att.cpu().numpy() - ev["attention"])[:, live_before]
            assert err.max() <= 1e-2 and err.mean() <= 1e-3
        np.testing.assert_array_equal(mask_out.cpu().numpy(), ev["mask"])
        m = ev["mask"].astype(bool)
        if m.any():
            assert np.abs(g_ys[m] - ev["step_scores"][m]).max() <= 1e-3
        n_ev += len(ev["evicted"]); n_fin += len(ev["finished"])
        _meta_equal(pool, ora_pool)
        vv = pool.vote_views()
        fin = np.flatnonzero(vv["finished"].cpu().numpy())
        assert sorted(fin.tolist()) == sorted(ora.finished)
    assert n_ev >= 2 and n_fin >= 2 and not ora.live()
    a, w, nf = pool.weighted_vote()
    assert int(nf.item()) == len(ora.finished)
    assert int(a.item()) == ora.vote(final_scores=pool.vote_views()["final_score"].cpu().numpy())
    assert pool.last_error()[1] == ora_pool.status == 0


def test_whole_run_in_one_call_against_the_oracle_replay():
    """algorithm1_run with ring-buffered inputs and a host check every 8 iterations; the oracle replays the run
    with the device's recorded score history."""
    n, iters, ring, seed = 24, 200, 7, 21
    cfg, vocab, eos, table, toks, answers, wx, wts, pool, ora_pool = _driver_case(seed, n, iters, 28, False, p_eos=0.03)
    gen = torch.Generator(device=DEV); gen.manual_seed(seed)
    rnd = lambda *shape: torch.randn(shape, generator=gen, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    q, k, v, h = rnd(ring, 2, n, 8, 128), rnd(ring, n, 1, 2, 2, 128), rnd(ring, n, 1, 2, 2, 128), rnd(ring, n, cfg.scorer_D)
    hist = torch.full((iters, n), float("nan"), dtype=torch.float32, device=DEV)
    res = pool.algorithm1_run(torch.from_numpy(toks).to(DEV), eos, table, torch.from_numpy(answers).to(DEV), q, k, v, h, wts,
                              1.0, -1.0, max_evictions=2, check_every=8, score_history=hist)
    assert res["live_left"] == 0 and res["iterations"] % 8 == 0 and res["iterations"] < iters
    ora = Algorithm1Oracle(ora_pool, n, *wx, vocab, eos, 1.0, -1.0, max_evictions=2)
    hx = h.float().cpu().numpy()
    hist_h = hist.cpu().numpy()
    used_iters = 0
    for i in range(res["iterations"]):
        if ora.live():
            used_iters = i + 1
        ora.iteration(toks[i], hx[i % ring], answers, rank_scores=hist_h[i])
    assert res["iterations"] - used_iters < 8                    # the host noticed at its next check
    _meta_equal(pool, ora_pool)
    assert res["n_finished"] == len(ora.finished) >= 2 and res["n_evicted"] == ora.n_evicted >= 2
    vv = pool.vote_views()
    assert sorted(np.flatnonzero(vv["finished"].cpu().numpy()).tolist()) == sorted(ora.finished)
    fs = vv["final_score"].cpu().numpy()
    for t, (s_, a_) in ora.finished.items():
        assert abs(fs[t] - s_) <= 1e-3 and int(vv["answer"][t].item()) == a_
    assert res["answer"] == ora.vote(final_scores=fs)
    assert pool.last_error()[1] == ora_pool.status == 0


def test_iteration_can_be_captured_in_a_cuda_graph_and_replayed():
    """algorithm1_iteration makes no host round trip, so one iteration per ring slot can be recorded as a CUDA graph and
    replayed; the replayed run ends in exactly the state and outputs of the eagerly launched one."""
    n, iters, ring, seed = 16, 48, 4, 31
    pools = []
    for _ in range(2):
        cfg, vocab, eos, table, toks, answers, wx, wts, pool, _ = _driver_case(seed, n, iters, 40, False, p_eos=0.03)
        pools.append((pool, wts))
    gen = torch.Generator(device=DEV); gen.manual_seed(seed)
    rnd = lambda *shape: torch.randn(shape, generator=gen, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    q, k, v, h = rnd(ring, 2, n, 8, 128), rnd(ring, n, 1, 2, 2, 128), rnd(ring, n, 1, 2, 2, 128), rnd(ring, n, cfg.scorer_D)
    ans = torch.from_numpy(answers).to(DEV)
    tok_slots = torch.zeros((ring, n), dtype=torch.int32, device=DEV)       # the graphs read the tokens from here
    toks_dev = torch.from_numpy(toks).to(DEV)
    outs = []
    for pool, wts in pools:
        outs.append(dict(att=torch.zeros((2, n, 8, 128), dtype=torch.float32, device=DEV),
                         ys=torch.zeros(n, dtype=torch.float32, device=DEV),
                         ts=torch.zeros(n, dtype=torch.float32, device=DEV)))

    def one(pi, slot):
        pool, wts = pools[pi]
        o = outs[pi]
        pool.algorithm1_iteration(tok_slots[slot], eos, table, ans, q[slot], k[slot], v[slot], h[slot], wts, 1.0, 0.5,
                                  max_evictions=1, attn_out=o["att"], step_scores_out=o["ys"], trace_scores_out=o["ts"])

    # first iterations eagerly on both pools (one-time set-up of the library happens outside any capture)
    for i in range(ring):
        tok_slots[i].copy_(toks_dev[i])
        one(0, i); one(1, i)
    torch.cuda.synchronize()
    graphs = []
    for slot in range(ring):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            one(1, slot)
        graphs.append(g)
    # capture recorded the launches without running them: pool 1 is still where pool 0 is
    for i in range(ring, iters):
        slot = i % ring
        tok_slots[slot].copy_(toks_dev[i])
        one(0, slot)
        hist0 = {k_: t.clone() for k_, t in outs[0].items()}
        graphs[slot].replay()
        torch.cuda.synchronize()
        for k_ in hist0:
            assert torch.equal(torch.nan_to_num(hist0[k_], nan=-7.0), torch.nan_to_num(outs[1][k_], nan=-7.0)), (i, k_)
    v0, v1 = pools[0][0].views(), pools[1][0].views()
    for name in ("block_table", "seq_lens", "live", "refcount", "free_count", "trace_scores"):
        assert torch.equal(v0[name], v1[name]), name
    fc = int(v0["free_count"].item())
    assert torch.equal(v0["free_list"][:fc], v1["free_list"][:fc])
    s0, s1 = pools[0][0].stats(), pools[1][0].stats()
    assert s0 == s1 and s0["live_traces"] < n
    assert pools[0][0].last_error() == (0, 0) and pools[1][0].last_error() == (0, 0)


def test_whole_run_with_recorded_iterations_equals_the_directly_launched_run():
    """algorithm1_run(use_graphs) replays one CUDA graph per ring slot; results, history and pool state are those of
    the run that launches every kernel itself."""
    n, iters, ring, seed = 24, 120, 5, 33
    runs = []
    for use_graphs in (False, True):
        cfg, vocab, eos, table, toks, answers, wx, wts, pool, _ = _driver_case(seed, n, iters, 28, False, p_eos=0.02)
        gen = torch.Generator(device=DEV); gen.manual_seed(seed)
        rnd = lambda *shape: torch.randn(shape, generator=gen, device=DEV, dtype=torch.float32).to(torch.bfloat16)
        q, k, v, h = rnd(ring, 2, n, 8, 128), rnd(ring, n, 1, 2, 2, 128), rnd(ring, n, 1, 2, 2, 128), rnd(ring, n, cfg.scorer_D)
        hist = torch.full((iters, n), float("nan"), dtype=torch.float32, device=DEV)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            res = pool.algorithm1_run(torch.from_numpy(toks).to(DEV), eos, table, torch.from_numpy(answers).to(DEV), q, k, v, h,
                                      wts, 1.0, 0.5, max_evictions=1, check_every=8, score_history=hist, use_graphs=use_graphs)
        torch.cuda.synchronize()
        runs.append((res, hist, pool))
    (r0, h0, p0), (r1, h1, p1) = runs
    assert r0 == r1 and r0["n_evicted"] >= 2 and r0["n_finished"] >= 2
    assert torch.equal(torch.nan_to_num(h0, nan=-7.0), torch.nan_to_num(h1, nan=-7.0))
    v0, v1 = p0.views(), p1.views()
    for name in ("block_table", "seq_lens", "live", "refcount", "free_count", "trace_scores"):
        assert torch.equal(v0[name], v1[name]), name
    assert p0.last_error() == (0, 0) and p1.last_error() == (0, 0)
