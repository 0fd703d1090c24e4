"""GPU parity at the benchmark configurations' full sizes, in the launch configuration bench.py times.

The pools are filled on the device (they are far too large to draw on the host); for a sample of traces the
stored K/V rows are read back through kv_pool_read_kv and the oracle computes those traces' outputs from the
very bytes the kernel read.  The prune test runs the memory-saturated configuration's five cycles with the
full-size bookkeeping (65,536 blocks, 64 traces, up to ~15.6k pages per trace; one layer of KV storage, which
the bookkeeping never looks at) against the oracle's pool, bit for bit.
"""
import math

import numpy as np
import pytest
import torch

from oracle import attention as OA
from oracle import scorer as OS
from paper_2601_09093_b200 import binding as B
from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W

from gpu_common import Twin

pytestmark = pytest.mark.gpu

ATT_MAX, ATT_MEAN = 1e-2, 1e-3


def _oracle_check(pool, cfg, layer, q, out, sample_traces):
    """out [T, Hq, d] of `layer` against the fp64 oracle on K/V rows read back from the pool, for the sampled traces."""
    v = pool.views()
    seq = v["seq_lens"].cpu().numpy()
    got = out.cpu().numpy().astype(np.float64)
    qx = q.float().cpu().numpy().astype(np.float64)
    worst_max, tot, cnt = 0.0, 0.0, 0
    for t in sample_traces:
        S = int(seq[t])
        K_ = np.empty((S, cfg.num_kv_heads, cfg.head_dim), dtype=np.float64)
        V_ = np.empty_like(K_)
        for h in range(cfg.num_kv_heads):
            k, vv = pool.read_kv(layer, h, v["block_table"][t], S)
            K_[:, h] = k.float().cpu().numpy(); V_[:, h] = vv.float().cpu().numpy()
        want = OA.dense_decode_attention(qx[t], K_, V_)
        err = np.abs(got[t] - want)
        worst_max = max(worst_max, float(err.max())); tot += float(err.sum()); cnt += err.size
    assert worst_max <= ATT_MAX and tot / cnt <= ATT_MEAN, (layer, worst_max, tot / cnt)


def _sampled_attention_parity(cfg, phys_layers, layer, sample_traces):
    suffix = W.suffix_lengths(cfg)
    T, P = cfg.n_traces, cfg.page_size
    pages = cfg.prefix_len // P + int(sum(-(-s // P) + 1 for s in suffix))
    max_pages = -(-(cfg.prefix_len + int(suffix.max())) // P) + 2
    cfg_pool = W.scaled(cfg, num_layers=phys_layers)
    pool = H.make_pool(cfg_pool, pages + 64, max_pages, T)
    if cfg.shuffle_pages:
        H.shuffle_free_list(pool, cfg.seed)
    H.fill_random_device(pool, cfg_pool, suffix, seed=cfg.seed, chunk_tokens=max(16, (1 << 28) // (T * cfg_pool.bytes_per_token)))
    v = pool.views()
    gen = torch.Generator(device="cuda"); gen.manual_seed(cfg.seed + 3)
    q_all = torch.randn((phys_layers, T, cfg.num_q_heads, cfg.head_dim), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    # all resident layers in one call, as the benchmark's step does: the checked layer's launch is then a programmatic
    # dependent of the layer before it
    out_all = pool.decode_attention_layers(0, q_all, v["block_table"], v["seq_lens"])
    plain = pool.decode_attention(layer, q_all[layer], v["block_table"], v["seq_lens"])
    assert torch.equal(out_all[layer], plain)
    q = q_all[layer]
    out = out_all[layer].cpu().numpy().astype(np.float64)
    assert pool.last_error() == (0, 0)
    seq = v["seq_lens"].cpu().numpy()
    assert np.array_equal(seq[:T], cfg.prefix_len + suffix)
    qx = q.float().cpu().numpy().astype(np.float64)
    worst_max, tot, cnt = 0.0, 0.0, 0
    for t in sample_traces:
        S = int(seq[t])
        K_ = np.empty((S, cfg.num_kv_heads, cfg.head_dim), dtype=np.float64)
        V_ = np.empty_like(K_)
        for h in range(cfg.num_kv_heads):
            k, vv = pool.read_kv(layer, h, v["block_table"][t], S)
            K_[:, h] = k.float().cpu().numpy(); V_[:, h] = vv.float().cpu().numpy()
        want = OA.dense_decode_attention(qx[t], K_, V_)
        err = np.abs(out[t] - want)
        worst_max = max(worst_max, float(err.max())); tot += float(err.sum()); cnt += err.size
    assert worst_max <= ATT_MAX and tot / cnt <= ATT_MEAN, (worst_max, tot / cnt)
    pool.close()


def test_c1_full_size_attention_sampled():
    """64 traces, 32/8 heads, 512 shared + U[4k,16k] tokens: shortest, longest and a few other traces."""
    s = W.suffix_lengths(W.C1)
    _sampled_attention_parity(W.C1, 2, 1, sorted({int(np.argmin(s)), int(np.argmax(s)), 0, 31, 63}))


def test_c4_full_size_attention_sampled():
    """128 traces, 64/8 heads (G = 8), 1024 shared + log-uniform 1k-24k tokens."""
    s = W.suffix_lengths(W.C4)
    _sampled_attention_parity(W.C4, 2, 1, sorted({int(np.argmin(s)), int(np.argmax(s)), 1, 64, 127}))


@pytest.mark.parametrize("layer", [0, 1])
def test_c2_long_traces_shuffled_pages_sampled(layer):
    """The long-trace shape (16k-32k tokens per trace, pages scattered over the pool): eight traces on each of two
    resident layers (layer 0's launch is the ordinary one of the layer-after-layer call, layer 1's its dependent)."""
    s = W.suffix_lengths(W.C2)
    _sampled_attention_parity(W.C2, 2, layer, sorted({int(np.argmin(s)), int(np.argmax(s)), 0, 5, 21, 32, 47, 63}))


def test_c3_attention_at_the_saturation_state_sampled():
    """The state the benchmark's headline is timed on: a 65,536-block pool (two resident layers), 64 traces grown
    from a 512-token shared prompt to just below the 95 % trigger (equal lengths, ~15.5k tokens), sized by the
    benchmark's own plan.  Both the layer-after-layer call and the plain per-layer call are checked against the
    oracle on nine traces (first, last, middle and others), all heads."""
    import bench
    steps_total = 40
    cfg, suffix, nb, max_pages, _ = bench.workload_plan("c3", 0, steps_total)
    assert nb == 65536 and cfg.n_traces == 64
    phys = 2
    cfg_pool = W.scaled(cfg, num_layers=phys)
    T = cfg.n_traces
    pool = H.make_pool(cfg_pool, nb, max_pages, T, max_score_rows=T)
    H.fill_random_device(pool, cfg_pool, suffix, seed=cfg.seed, chunk_tokens=max(16, (1 << 28) // (T * cfg_pool.bytes_per_token)))
    v = pool.views()
    st = pool.stats()
    limit = math.floor(float(np.float32(cfg.threshold)) * nb)
    assert st["live_traces"] == T and st["used"] + T <= limit < st["used"] + T * (steps_total // cfg.page_size + 4)
    # one more token per trace, as a decode step appends it
    gen = torch.Generator(device="cuda"); gen.manual_seed(cfg.seed + 5)
    rnd = lambda *shape: torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    ids = torch.arange(T, dtype=torch.int32, device="cuda")
    pool.append_kv(ids, 1, rnd(T, 1, phys, cfg.num_kv_heads, cfg.head_dim), rnd(T, 1, phys, cfg.num_kv_heads, cfg.head_dim))
    q_all = rnd(phys, T, cfg.num_q_heads, cfg.head_dim)
    out_all = pool.decode_attention_layers(0, q_all, v["block_table"], v["seq_lens"])
    sample = [0, 1, 7, 20, 31, 32, 45, 62, 63]
    for layer in range(phys):
        plain = pool.decode_attention(layer, q_all[layer], v["block_table"], v["seq_lens"])
        assert torch.equal(out_all[layer], plain)
        _oracle_check(pool, cfg, layer, q_all[layer], out_all[layer], sample)
    pid, n = pool.prune_if_saturated(None, cfg.threshold, cfg.keep_frac)
    assert int(n.item()) == 0                                       # just below the trigger: nothing fires
    assert pool.last_error() == (0, 0)
    pool.close()


def _scorer_rows_sampled(D, m, rows, sample_rows):
    """score_steps on `rows` rows that all end a step (hidden states drawn on the device); the oracle scores the
    sampled rows from the very bf16 values the kernel read."""
    cfg = W.scaled(W.C1, scorer_D=D, scorer_m=m, seed=4242 + D + m)
    T = 64
    pool = H.make_pool(W.scaled(cfg, num_layers=1), 8, 4, T, max_score_rows=rows)
    (W1b, W1x), (b1b, b1x), (w2b, w2x), b2 = W.scorer_weights(cfg, bias_std=0.05)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16"), H.to_device(b1b, "bf16"), H.to_device(w2b, "bf16"), b2, B.STEP_BF16)
    gen = torch.Generator(device="cuda"); gen.manual_seed(cfg.seed)
    hid = torch.randn((rows, D), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    mask = torch.ones(rows, dtype=torch.uint8, device="cuda")
    rt = (torch.arange(rows, device="cuda") % T).to(torch.int32)
    got = pool.score_steps(hid, mask, rt, wts).cpu().numpy()
    info = pool.score_launch_info()
    assert info["n_rows"] == rows and info["tc_units"] > 0           # the tensor-core kernel scored them
    assert np.isfinite(got).all()
    idx = np.asarray(sorted(set(int(r) for r in sample_rows if 0 <= r < rows)))
    hx = hid[torch.from_numpy(idx).cuda()].float().cpu().numpy().astype(np.float64)
    want = OS.score_steps(hx, np.ones(len(idx), dtype=np.uint8), W1x, b1x, w2x, b2)
    assert np.abs(got[idx] - want).max() <= 1e-3, float(np.abs(got[idx] - want).max())
    # running means: every trace's mean over its rows, from the GPU's own scores
    ts = OS.TraceScores(T)
    ts.update(got, np.ones(rows, dtype=np.uint8), row_trace=(np.arange(rows) % T))
    np.testing.assert_allclose(pool.views()["trace_scores"].cpu().numpy(), ts.scores(), atol=1e-4)
    assert pool.last_error() == (0, 0)
    pool.close()
    return info


@pytest.mark.parametrize("D,m", [(4096, 512), (5120, 1024)])
def test_scorer_65536_step_end_rows_sampled(D, m):
    """The launch the batched-scorer benchmark times: 65,536 rows, 256-row x 256-unit items with two accumulators,
    the last round cut into 128-row items.  With 148 CTAs the 256-row items cover rows [0, 56,832) and the 128-row
    items the rest; the sample takes rows of both halves of the first and of a late 256-row item, rows on either side
    of that boundary, rows of the 128-row items, the very last rows, and 64 rows spread over the launch."""
    rows = 65536
    sample = (list(range(0, 40)) + list(range(128, 168)) + list(range(56832 - 256, 56832 - 216)) + list(range(56832 - 40, 56832 + 88))
              + list(range(60000, 60016)) + list(range(rows - 72, rows)) + list(range(517, rows, 1021)))
    info = _scorer_rows_sampled(D, m, rows, sample)
    assert info["tc_units"] == 256


def test_scorer_d5120_m512_sampled():
    """The 14B-class model width with the paper's 512-unit scorer (hidden 5120): a 20,000-row launch."""
    rows = 20000
    sample = list(range(0, 48)) + list(range(128, 176)) + list(range(rows - 80, rows)) + list(range(311, rows, 157))
    _scorer_rows_sampled(5120, 512, rows, sample)


@pytest.mark.parametrize("n_traces,threshold", [(64, 0.95), (16, 0.5), (16, 0.9), (32, 0.5), (32, 0.7), (32, 0.9)])
def test_c3_prune_cycles_full_size_bookkeeping(n_traces, threshold):
    """The memory-saturated configuration's prune cycles with the full-size bookkeeping, at the benchmark's default
    (64 traces, 95 %) and at the sampling budgets N = 16 / 32 and memory budgets 0.5 - 0.9 its sweeps time: every
    cycle halves the live set until two traces share the pool."""
    cfg = W.scaled(W.C3, num_layers=1, n_traces=n_traces, threshold=threshold)
    T, nb, P = cfg.n_traces, W.C3.num_blocks, cfg.page_size
    limit = math.floor(float(np.float32(cfg.threshold)) * nb)
    max_pages = cfg.prefix_len // P + limit // 4 + 64
    tw = Twin(cfg, nb, max_pages, T, store_payload=False, max_score_rows=T)
    ids, oids = tw.fork(T, cfg.prefix_len)
    assert ids == oids
    full = W.C3                                                  # the scorer of the full configuration
    (W1b, W1x), (b1b, b1x), (w2b, w2x), b2 = W.scorer_weights(full, bias_std=0.05)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16"), H.to_device(b1b, "bf16"), H.to_device(w2b, "bf16"), b2, B.STEP_BF16)
    ts = OS.TraceScores(T)
    live = list(ids)
    cycles = 0
    while len(live) > 2:
        cyc = cycles
        cycles += 1
        # grow every live trace to the page boundary at which the pool reaches the trigger
        used = tw.gpu.stats()["used"]
        assert used == tw.ora.used
        S = int(tw.ora.seq_lens[live[0]])
        n_tok = (-(-S // P) + (limit - used) // len(live)) * P - S
        while n_tok > 0:
            c = min(n_tok, 2048)
            assert all(tw.append(live, c))
            n_tok -= c
        assert tw.ora.saturated(cfg.threshold)
        hb, hx = W.normal(cfg.seed, W.TID_HID, (T, full.scorer_D), "bf16", sub=cyc)
        mask = np.zeros(T, dtype=np.uint8); mask[live] = 1
        g = tw.gpu.score_steps(H.to_device(hb, "bf16"), torch.from_numpy(mask).cuda(), None, wts).cpu().numpy()
        want = OS.score_steps(hx, mask, W1x, b1x, w2x, b2)
        assert np.abs(g[mask == 1] - want[mask == 1]).max() <= 1e-3
        ts.update(g, mask)
        scores = tw.gpu.views()["trace_scores"].cpu().numpy()
        np.testing.assert_allclose(scores[live], ts.scores()[live], atol=1e-6)
        pid, n = tw.gpu.prune_if_saturated(None, cfg.threshold, cfg.keep_frac)
        got = pid[: int(n.item())].cpu().tolist()
        assert got == tw.ora.prune_if_saturated(scores, cfg.threshold, cfg.keep_frac, on_evict=ts.clear)
        assert len(got) == len(live) // 2
        live = [t for t in live if t not in got]
        tw.assert_meta_equal()
        assert all(tw.append(live, 1))                           # no waiting queue: every survivor is scheduled
        assert tw.status() == (0, 0)
    assert len(live) == 2 and (1 << cycles) * 2 == T
    tw.assert_meta_equal()
