"""decode_attention_static: the entry point for callers that may not allocate device memory.

Some hosts of this library (a plug-in inside another framework's memory pool, a serving loop that
forbids allocator calls once it is running) cannot give the attention kernel scratch memory.  For
them the library carries a fixed scratch array of its own.  This test calls that entry point through
the C ABI twice in a row - the second time on different inputs, so that whatever the first call left
in the shared array would show - and checks each result against the ordinary entry point.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from oracle import attention as OA
from paper_2601_09093_b200 import binding as B
from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W

pytestmark = pytest.mark.gpu

ATT_MAX, ATT_MEAN = 1e-2, 1e-3          # the tolerances of the other attention parity tests


def _pool_with_traces(cfg, suffix, seed):
    P = cfg.page_size
    nb = int(sum(-(-(cfg.prefix_len + s) // P) for s in suffix)) + 8
    pool = H.make_pool(cfg, nb, -(-(cfg.prefix_len + int(max(suffix))) // P) + 2, len(suffix))
    H.fill_random_device(pool, cfg, np.asarray(suffix), seed=seed, chunk_tokens=512)
    return pool


def _compare(pool, cfg, n, q_sub):
    v = pool.views()
    qb, _ = W.normal(cfg.seed, W.TID_Q, (n, cfg.num_q_heads, cfg.head_dim), "bf16", sub=q_sub)
    q = H.to_device(qb, "bf16")
    want = pool.decode_attention(0, q, v["block_table"][:n], v["seq_lens"][:n])
    out = torch.full_like(want, float("nan"))           # caller-owned output; the call allocates nothing
    pool.decode_attention_static(0, q, v["block_table"][:n], v["seq_lens"][:n], out)
    torch.cuda.synchronize()
    err = (out.double() - want.double()).abs()
    assert torch.isfinite(out).all()
    assert err.max().item() <= ATT_MAX and err.mean().item() <= ATT_MEAN, (err.max().item(), err.mean().item())
    assert pool.last_error() == (0, 0)


def test_static_scratch_matches_regular_entry_point_twice_in_a_row():
    cfg = W.scaled(W.C1, n_traces=7, prefix_len=48)
    pool = _pool_with_traces(cfg, [0, 1, 17, 900, 2600, 333, 4100], seed=11)
    _compare(pool, cfg, 7, q_sub=1)
    # second call: other queries, fewer traces and another split of the KV stream, so stale partials
    # of the first call sit in slots this call also uses
    pool.set_attention_config(grid_ctas=5)
    _compare(pool, cfg, 5, q_sub=2)
    # and a different pool on the same device shares the same array
    pool2 = _pool_with_traces(W.scaled(W.C1, n_traces=3, prefix_len=16, num_q_heads=64), [700, 20, 1500], seed=12)
    _compare(pool2, W.scaled(W.C1, n_traces=3, prefix_len=16, num_q_heads=64), 3, q_sub=3)


def test_static_call_allocates_nothing_and_agrees_with_the_oracle():
    """What the entry point is for: after the first call on the device (which looks up the array's address) a
    call leaves the driver's free memory and torch's allocator exactly as it found them.  The result of that
    call is also compared with the CPU oracle directly, on K/V rows read back from the pool."""
    cfg = W.scaled(W.C1, n_traces=5, prefix_len=32)
    suffix = [3, 700, 0, 1900, 65]
    pool = _pool_with_traces(cfg, suffix, seed=21)
    v = pool.views()
    qb, qx = W.normal(cfg.seed, W.TID_Q, (5, cfg.num_q_heads, cfg.head_dim), "bf16", sub=9)
    q = H.to_device(qb, "bf16")
    out = torch.empty((5, cfg.num_q_heads, cfg.head_dim), dtype=torch.float32, device="cuda")
    bt, sl = v["block_table"][:5], v["seq_lens"][:5]
    pool.decode_attention_static(0, q, bt, sl, out)              # first call on this device: set-up included
    torch.cuda.synchronize()
    free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    out.fill_(float("nan"))
    pool.decode_attention_static(0, q, bt, sl, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    got = out.cpu().numpy().astype(np.float64)
    for t in range(5):
        S = cfg.prefix_len + suffix[t]
        K_ = np.empty((S, cfg.num_kv_heads, cfg.head_dim)); V_ = np.empty_like(K_)
        for h in range(cfg.num_kv_heads):
            k, vv = pool.read_kv(0, h, v["block_table"][t], S)
            K_[:, h] = k.float().cpu().numpy(); V_[:, h] = vv.float().cpu().numpy()
        err = np.abs(got[t] - OA.dense_decode_attention(qx[t].astype(np.float64), K_, V_))
        assert err.max() <= ATT_MAX and err.mean() <= ATT_MEAN
    assert pool.last_error() == (0, 0)


def test_static_scratch_rejects_more_sequences_than_its_counters_hold():
    """n > 2048 traces, or more than 16,384 (trace, KV head) sequences, do not fit the fixed array: STEP_ERR_CAPACITY
    before anything is launched, the output untouched."""
    one_head = W.scaled(W.C1, n_traces=2049, prefix_len=0, num_q_heads=4, num_kv_heads=1)
    pool = H.make_pool(one_head, 8, 2, 2049)
    v = pool.views()
    q = torch.zeros((2049, 4, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.full((2049, 4, 128), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(B.StepError) as e:
        pool.decode_attention_static(0, q, v["block_table"], v["seq_lens"], out)
    assert e.value.code == 4
    many_heads = W.scaled(W.C1, n_traces=1100, prefix_len=0, num_q_heads=16, num_kv_heads=16)     # 17,600 sequences
    pool2 = H.make_pool(many_heads, 8, 2, 1100)
    v2 = pool2.views()
    q2 = torch.zeros((1100, 16, 128), dtype=torch.bfloat16, device="cuda")
    out2 = torch.full((1100, 16, 128), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(B.StepError) as e:
        pool2.decode_attention_static(0, q2, v2["block_table"], v2["seq_lens"], out2)
    assert e.value.code == 4
    torch.cuda.synchronize()
    assert (out == 7.0).all() and (out2 == 7.0).all()
    pool2.decode_attention_static(0, q2[:1024], v2["block_table"][:1024], v2["seq_lens"][:1024], out2[:1024])   # 16,384: fits
    torch.cuda.synchronize()
    assert (out2[:1024] == 0.0).all()                            # empty traces give zeros


def test_static_scratch_rejects_what_does_not_fit():
    big_group = W.scaled(W.C1, n_traces=1, prefix_len=16, num_q_heads=128)      # 16 query heads per KV head
    pool = _pool_with_traces(big_group, [40], seed=13)
    v = pool.views()
    q = torch.zeros((1, 128, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 128, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(B.StepError) as e:
        pool.decode_attention_static(0, q, v["block_table"][:1], v["seq_lens"][:1], out)
    assert e.value.code == 4                                                      # STEP_ERR_CAPACITY
    fp32_pool = H.make_pool(W.C0, 8, 4)
    with pytest.raises(B.StepError) as e:
        fp32_pool.decode_attention_static(0, out, v["block_table"][:1], v["seq_lens"][:1], out)
    assert e.value.code == 1                                                      # STEP_ERR_INVALID_ARG
