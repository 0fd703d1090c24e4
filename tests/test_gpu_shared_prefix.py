"""decode_attention_shared_prefix against the oracle, and against decode_attention on pools whose traces share
their prompt pages."""
import numpy as np
import pytest
import torch

from oracle import attention as OA
from paper_2601_09093_b200 import binding as B
from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W

from gpu_common import Twin, exact_f32, attention_errors

pytestmark = pytest.mark.gpu
ATT_MAX, ATT_MEAN = 1e-2, 1e-3


def _build(cfg, suffix, extra_blocks=8, max_traces=None):
    P = cfg.page_size
    n = len(suffix)
    pages = int(sum(-(-(cfg.prefix_len + int(s)) // P) for s in suffix)) + extra_blocks
    tw = Twin(cfg, pages, -(-(cfg.prefix_len + int(max(suffix))) // P) + 2, max_traces or n)
    ids, oids = tw.fork(n, cfg.prefix_len)
    assert ids == oids
    for sel, inc in H.ragged_append_plan(np.asarray(suffix)):
        if inc > 0:
            assert all(tw.append([ids[i] for i in sel], inc))
    return tw, ids


def _compare(tw, cfg, n, pp, prefix_row, layer=0, seq_lens=None):
    v = tw.gpu.views()
    qb, qx = W.normal(cfg.seed, W.TID_Q, (n, cfg.num_q_heads, cfg.head_dim), cfg.dtype, sub=77 + layer)
    qd = H.to_device(qb, cfg.dtype)
    sl_dev = v["seq_lens"][:n] if seq_lens is None else torch.tensor(seq_lens, dtype=torch.int32, device=qd.device)
    sl_ora = tw.ora.seq_lens[:n] if seq_lens is None else np.asarray(seq_lens)
    prefix_dev = v["block_table"][prefix_row, :pp].contiguous()
    got = exact_f32(tw.gpu.decode_attention_shared_prefix(layer, qd, v["block_table"][:n], sl_dev, prefix_dev, pp))
    want, short = OA.paged_decode_attention_shared_prefix(qx, tw.ora.k_pages[layer], tw.ora.v_pages[layer],
                                                          tw.ora.block_table[:n], sl_ora, tw.ora.block_table[prefix_row, :pp])
    mx, mean = attention_errors(got, want)
    assert mx <= ATT_MAX and mean <= ATT_MEAN, (mx, mean)
    return got, qd, short


@pytest.mark.parametrize("hq,hkv,n,prefix_len", [
    (32, 8, 13, 100),      # G = 4: bundles of 4 traces, the last one ragged; 6 shared pages + a private partial page
    (64, 8, 7, 96),        # G = 8: bundles of 2; the prompt fills its pages exactly
    (40, 8, 10, 200),      # G = 5: bundles of 3 traces use 15 of the 16 rows
    (32, 2, 5, 64),        # G = 16: one trace per bundle, both row halves of the tile
    (8, 8, 20, 48),        # G = 1: 16 traces per bundle
])
def test_shared_prefix_matches_oracle_and_plain_kernel(hq, hkv, n, prefix_len):
    cfg = W.scaled(W.C1, n_traces=n, num_q_heads=hq, num_kv_heads=hkv, prefix_len=prefix_len, seed=4200 + hq + n)
    g = W.rng(cfg.seed, W.TID_LEN)
    suffix = g.integers(0, 300, size=n)
    suffix[0] = 0                                    # a trace that holds the prompt and nothing else
    tw, ids = _build(cfg, suffix)
    pp = prefix_len // cfg.page_size
    got, qd, short = _compare(tw, cfg, n, pp, prefix_row=1)
    assert short == [] and tw.status() == (0, 0)
    v = tw.gpu.views()
    plain = exact_f32(tw.gpu.decode_attention(0, qd, v["block_table"][:n], v["seq_lens"][:n]))
    assert np.abs(got - plain).max() <= 2e-3        # the two kernels round differently (split points differ)


def test_long_prompt_many_traces_prefix_pass_is_split_and_merged():
    cfg = W.scaled(W.C1, n_traces=64, prefix_len=4096 + 7, seed=4301)
    suffix = W.rng(cfg.seed, W.TID_LEN).integers(1, 200, size=64)
    tw, ids = _build(cfg, suffix)
    pp = 4096 // 16
    _compare(tw, cfg, 64, pp, prefix_row=63)
    # evict a few traces (their rows become empty): zeros for them, the rest unchanged
    tw.gpu.release_traces(torch.tensor([0, 5, 6, 7, 63], dtype=torch.int32, device="cuda:0"))
    for t in (0, 5, 6, 7, 63):
        tw.ora.release_trace(t)
    got, _, short = _compare(tw, cfg, 64, pp, prefix_row=1)
    assert short == [] and np.all(got[[0, 5, 6, 7, 63]] == 0)
    assert tw.status() == (0, 0)
    tw.assert_meta_equal()


def test_rows_that_do_not_share_use_the_given_blocks_and_short_rows_are_flagged():
    cfg = W.scaled(W.C1, n_traces=6, prefix_len=64, seed=4302)
    tw, ids = _build(cfg, [40, 3, 90, 17, 0, 55], extra_blocks=16, max_traces=8)
    # a second, unrelated problem in the same pool: its pages differ from the first one's
    ids2, _ = tw.fork(2, 64)
    tw.append(ids2, 30)
    n = 8
    got, qd, short = _compare(tw, cfg, n, 4, prefix_row=0)          # rows 6, 7 read problem 1's prompt all the same
    assert short == []
    sl = tw.ora.seq_lens[:n].copy(); sl[2] = 50; sl[3] = 0
    got, _, short = _compare(tw, cfg, n, 4, prefix_row=0, seq_lens=sl)
    assert short == [2] and np.all(got[2] == 0) and np.all(got[3] == 0)
    assert tw.status()[0] == 1 << 1       # STEP_ERR_INVALID_ARG


def test_shared_prefix_argument_checks():
    cfg = W.scaled(W.C0, prefix_len=16)
    tw = Twin(cfg, 8, 4, 2, store_payload=False)                     # fp32 pool: the call is refused
    tw.fork(2, 16)
    v = tw.gpu.views()
    q = torch.zeros(2, cfg.num_q_heads, cfg.head_dim, device="cuda:0")
    with pytest.raises(B.StepError):
        tw.gpu.decode_attention_shared_prefix(0, q, v["block_table"], v["seq_lens"], v["block_table"][0], 1)
    out = tw.gpu.decode_attention_shared_prefix(0, q, v["block_table"], v["seq_lens"], v["block_table"][0], 0)
    assert torch.isfinite(out).all()                                  # prefix_pages = 0 is the plain call
