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


def test_c2_long_traces_shuffled_pages_sampled():
    """The long-trace shape (16k-32k tokens per trace, pages scattered over the pool) on two resident layers."""
    s = W.suffix_lengths(W.C2)
    _sampled_attention_parity(W.C2, 2, 1, sorted({int(np.argmin(s)), int(np.argmax(s)), 5}))


def test_c3_five_prune_cycles_full_size_bookkeeping():
    cfg = W.scaled(W.C3, num_layers=1)
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
    for cyc in range(5):
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
    assert len(live) == 2
    tw.assert_meta_equal()
