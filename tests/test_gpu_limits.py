"""GPU parity at the edges of what the kernels are built for: largest trace counts of the fast paths and the
fallbacks just beyond them, full block tables, lists longer than the shared-memory staging, the paper's third
scorer width."""
import numpy as np
import pytest
import torch

from oracle import attention as OA
from oracle import scorer as OS
from paper_2601_09093_b200 import binding as B
from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W

from gpu_common import Twin, exact_f32, attention_errors

pytestmark = pytest.mark.gpu


def _many_short_traces(n, seed):
    """n traces sharing a 16-token prompt, 0-40 further tokens each (some stay at the bare prompt)."""
    cfg = W.scaled(W.C1, n_traces=n, num_q_heads=8, num_kv_heads=2, prefix_len=16, seed=seed)
    tw = Twin(cfg, n * 3 + 8, 4, n)
    ids, _ = tw.fork(n, 16)
    extra = W.rng(seed, W.TID_LEN).integers(0, 41, size=n)
    for sel, inc in H.ragged_append_plan(extra):
        assert all(tw.append([ids[i] for i in sel], inc))
    return cfg, tw


@pytest.mark.parametrize("n", [2048, 2049])
def test_attention_at_and_beyond_the_tensor_core_kernels_trace_limit(n):
    """2048 rows is the most the tensor-core kernel takes in one call; 2049 goes to the scalar kernel."""
    cfg, tw = _many_short_traces(n, 31)
    qb, qx = W.normal(cfg.seed, W.TID_Q, (n, 8, 128), "bf16")
    v = tw.gpu.views()
    got = exact_f32(tw.gpu.decode_attention(0, H.to_device(qb, "bf16"), v["block_table"], v["seq_lens"]))
    want = OA.paged_decode_attention(qx, tw.ora.k_pages[0], tw.ora.v_pages[0], tw.ora.block_table, tw.ora.seq_lens)
    mx, mean = attention_errors(got, want)
    assert mx <= 1e-2 and mean <= 1e-3
    assert tw.status() == (0, 0)


def test_full_block_table_and_capacity_errors():
    """A trace that fills its block table to the last slot attends over all of it; one more token is refused."""
    cfg = W.scaled(W.C1, n_traces=2, num_q_heads=8, num_kv_heads=2, prefix_len=16)
    tw = Twin(cfg, 24, 8, 2)                                     # 8 pages = 128 tokens per trace at most
    ids, _ = tw.fork(2, 16)
    assert all(tw.append(ids, 112))
    assert tw.append(ids[:1], 1) == [False]                       # table full: skipped and flagged on both sides
    mask, omask = tw.status()
    assert mask == omask == 1 << 4
    tw.assert_meta_equal()
    qb, qx = W.normal(cfg.seed, W.TID_Q, (2, 8, 128), "bf16")
    v = tw.gpu.views()
    got = exact_f32(tw.gpu.decode_attention(0, H.to_device(qb, "bf16"), v["block_table"], v["seq_lens"]))
    want = OA.paged_decode_attention(qx, tw.ora.k_pages[0], tw.ora.v_pages[0], tw.ora.block_table, tw.ora.seq_lens)
    mx, mean = attention_errors(got, want)
    assert mx <= 1e-2 and mean <= 1e-3


def test_prune_list_longer_than_the_shared_memory_staging():
    """2048 live traces, three quarters evicted: the eviction list (1536) exceeds what the release stages in shared
    memory, so the offsets come from global memory; free list and tables must still match the oracle bit for bit."""
    n = 2048
    cfg = W.scaled(W.C0, n_traces=n, prefix_len=16)
    tw = Twin(cfg, n * 3 + 8, 4, n, store_payload=False)
    ids, _ = tw.fork(n, 16)
    extra = W.rng(7, W.TID_LEN).integers(1, 33, size=n)
    for sel, inc in H.ragged_append_plan(extra):
        assert all(tw.append([ids[i] for i in sel], inc))
    scores = W.rng(7, W.TID_ANS).random(n).astype(np.float32)
    scores[::97] = scores[5]                                       # ties
    pid, npr = tw.gpu.prune_if_saturated(torch.from_numpy(scores).cuda(), 0.01, 0.25)
    got = pid[: int(npr.item())].cpu().tolist()
    assert got == tw.ora.prune_if_saturated(scores, 0.01, 0.25) and len(got) == 1536
    tw.assert_meta_equal()
    assert tw.status() == (0, 0)


@pytest.mark.parametrize("n", [5000, 3000])
def test_append_list_longer_than_one_launch(n):
    """Thousands of traces in one append_kv call: the list is served in several launches, in list order.  A pool of
    5000 traces takes the two-launch form of append_kv (allocation kernel, then the rows), one of 3000 the one-launch
    form; both must follow the serial rule when the free list runs short in the middle of a list, and catch repeats."""
    cfg = W.scaled(W.C0, n_traces=n, prefix_len=16)
    tw = Twin(cfg, n + 64, 3, n, store_payload=False)
    ids, _ = tw.fork(n, 16)
    order = W.rng(3, W.TID_PERM).permutation(n).tolist()          # not ascending: allocation follows the list
    assert all(tw.append(order, 1))
    tw.assert_meta_equal()
    assert tw.status() == (0, 0)
    # 63 blocks are left and every trace wants one more page: the first 63 of the list get theirs
    served = tw.append(order, 16)
    assert sum(served) == 63 and all(served[:63])
    tw.assert_meta_equal()
    assert tw.status() == (1 << 2, 1 << 2)                        # STEP_ERR_NO_BLOCKS
    # repeats inside one launch's part of the list are served once
    short = order[100:140] + order[100:120]
    z = torch.zeros((len(short), 1, cfg.num_layers, cfg.num_kv_heads, cfg.head_dim), dtype=tw.gpu.torch_dtype, device="cuda")
    tw.gpu.append_kv(torch.tensor(short, dtype=torch.int32, device="cuda"), 1, z, z)
    tw.ora.append_kv(order[100:140], 1)
    tw.assert_meta_equal()
    assert tw.gpu.last_error()[1] == 1 << 3                        # STEP_ERR_BAD_TRACE


def test_scorer_width_2560_on_the_tensor_cores():
    """The paper's smallest hidden size (2560, scorer width 512): 40 k-chunks, a count that is not a power of two."""
    cfg = W.scaled(W.C1, scorer_D=2560, scorer_m=512)
    M, T = 700, 64
    pool = H.make_pool(cfg, 8, 4, T, max_score_rows=M)
    (W1b, W1x), (b1b, b1x), (w2b, w2x), b2 = W.scorer_weights(cfg, bias_std=0.05)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16"), H.to_device(b1b, "bf16"), H.to_device(w2b, "bf16"), b2, B.STEP_BF16)
    hb, hx = W.normal(cfg.seed, W.TID_HID, (M, 2560), "bf16")
    mask = W.boundary_mask(cfg, M, density=0.5)
    rt = torch.from_numpy((np.arange(M) % T).astype(np.int32)).cuda()
    got = pool.score_steps(H.to_device(hb, "bf16"), torch.from_numpy(mask).cuda(), rt, wts).cpu().numpy()
    assert pool.score_launch_info()["tc_units"] == 64
    want = OS.score_steps(hx, mask, W1x, b1x, w2x, b2)
    assert np.abs(got[mask == 1] - want[mask == 1]).max() <= 1e-3
    assert OS.scorer_flops(512, 2560) == 2622464                  # the appendix's 2m(d+1)
    assert pool.last_error() == (0, 0)


def test_scorer_width_8192_runs_on_the_tensor_cores_only():
    """D = 8192 is more than the CUDA-core kernel can stage; the tensor-core kernel takes it, the other path says no."""
    cfg = W.scaled(W.C1, scorer_D=8192, scorer_m=256)
    M, T = 300, 64
    pool = H.make_pool(cfg, 8, 4, T, max_score_rows=M)
    (W1b, W1x), (b1b, b1x), (w2b, w2x), b2 = W.scorer_weights(cfg, std=0.03, bias_std=0.05)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16"), H.to_device(b1b, "bf16"), H.to_device(w2b, "bf16"), b2, B.STEP_BF16)
    hb, hx = W.normal(cfg.seed, W.TID_HID, (M, 8192), "bf16")
    mask = W.boundary_mask(cfg, M, density=0.3)
    rt = torch.from_numpy((np.arange(M) % T).astype(np.int32)).cuda()
    got = pool.score_steps(H.to_device(hb, "bf16"), torch.from_numpy(mask).cuda(), rt, wts).cpu().numpy()
    want = OS.score_steps(hx, mask, W1x, b1x, w2x, b2)
    assert np.abs(got[mask == 1] - want[mask == 1]).max() <= 1e-3
    pool.set_scorer_config(-1, 0)
    with pytest.raises(B.StepError) as e:
        pool.score_steps(H.to_device(hb, "bf16"), torch.from_numpy(mask).cuda(), rt, wts)
    assert e.value.code == 1


def test_shared_prefix_attention_at_the_trace_limit_and_beyond():
    """2048 traces sharing one prompt page (G = 4: 512 bundles of 4) through decode_attention_shared_prefix; one trace
    more is refused with nothing launched."""
    n = 2048
    cfg, tw = _many_short_traces(n, 37)
    qb, qx = W.normal(cfg.seed, W.TID_Q, (n, 8, 128), "bf16")
    v = tw.gpu.views()
    prefix = v["block_table"][5, :1].contiguous()
    got = exact_f32(tw.gpu.decode_attention_shared_prefix(0, H.to_device(qb, "bf16"), v["block_table"], v["seq_lens"], prefix, 1))
    want, short = OA.paged_decode_attention_shared_prefix(qx, tw.ora.k_pages[0], tw.ora.v_pages[0], tw.ora.block_table,
                                                          tw.ora.seq_lens, tw.ora.block_table[5, :1])
    mx, mean = attention_errors(got, want)
    assert short == [] and mx <= 1e-2 and mean <= 1e-3
    assert tw.status() == (0, 0)
    cfg2, tw2 = _many_short_traces(2049, 38)
    v2 = tw2.gpu.views()
    q2 = torch.zeros((2049, 8, 128), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(B.StepError):
        tw2.gpu.decode_attention_shared_prefix(0, q2, v2["block_table"], v2["seq_lens"], v2["block_table"][0, :1].contiguous(), 1)
    with pytest.raises(B.StepError):                              # more shared pages than a block-table row holds
        tw.gpu.decode_attention_shared_prefix(0, H.to_device(qb, "bf16"), v["block_table"], v["seq_lens"], prefix, 5)


def test_train_step_smallest_shapes():
    """One hidden unit, one input dimension, three samples: the training kernels' tiles are almost entirely padding."""
    from oracle import training as OT
    H_ = np.array([[0.5], [-1.0], [2.0]]); y = np.array([1.0, 0.0, 1.0])
    params = [np.array([[0.7]]), np.array([0.1]), np.array([-0.4]), np.array([0.05])]
    opt = OT.Adam(params)
    tr = B.ScorerTrainer(torch.tensor([[0.7]], device="cuda:0"), torch.tensor([0.1], device="cuda:0"),
                         torch.tensor([-0.4], device="cuda:0"), 0.05, batch=3, pos_weight=0.5)
    Hd = torch.tensor(H_, dtype=torch.float32, device="cuda:0"); yd = torch.tensor(y, dtype=torch.float32, device="cuda:0")
    for _ in range(4):
        lg = float(tr.step(Hd, yd).cpu()[0])
        lo, params = OT.train_step(H_, y, params, opt, 0.5)
        assert abs(lg - lo) <= 2e-5
    for ref, got in zip(params, (tr.W1, tr.b1, tr.w2, tr.b2)):
        np.testing.assert_allclose(got.cpu().numpy().reshape(ref.shape), ref, rtol=0, atol=5e-6)


def test_a_page_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    """The bounded wait of the attention kernel, made to run out on purpose in the one safe way: with the limit set to
    zero a warp gives up on a page that has not landed by the time it first looks - while the copy itself is healthy
    and lands a microsecond later.  The warp must flag STEP_ERR_TIMEOUT, wait out the copies it has in flight (full
    limit) and leave; the call returns, nothing hangs, and the very next call on the same pool - no reset: nothing of
    the kernel's state outlives a launch - gives correct results."""
    from oracle import attention as OA
    cfg = W.scaled(W.C1, n_traces=6, prefix_len=32, seed=909)
    suffix = [8000, 64, 6000, 0, 333, 7000]
    P = cfg.page_size
    nb = int(sum(-(-(cfg.prefix_len + s) // P) for s in suffix)) + 8
    tw = Twin(cfg, nb, -(-(cfg.prefix_len + max(suffix)) // P) + 2, 6)

    def fill():
        ids, oids = tw.fork(6, cfg.prefix_len)
        assert ids == oids
        for sel, inc in H.ragged_append_plan(np.asarray(suffix)):
            assert all(tw.append([ids[i] for i in sel], inc))

    fill()
    qb, qx = W.normal(cfg.seed, W.TID_Q, (6, 32, 128), "bf16")
    q = H.to_device(qb, "bf16")
    v = tw.gpu.views()
    # (about twenty pages per warp on every SM: with the memory system saturated a copy takes microseconds and a
    # page's arithmetic a fraction of one, so warps are certain to look at pages that have not landed yet)
    tw.gpu.set_wait_limit_ns(0)
    out = tw.gpu.decode_attention(0, q, v["block_table"][:6], v["seq_lens"][:6])       # returns; results undefined
    torch.cuda.synchronize()
    code, mask = tw.gpu.last_error()
    assert mask & (1 << 6), mask                                                       # STEP_ERR_TIMEOUT
    # back to the normal limit: results as the oracle's, with every way of handing out the pages
    tw.gpu.set_wait_limit_ns(2_000_000_000)
    for sixteenths, chunk in ((4, 16), (12, 1), (0, 0)):
        tw.gpu.set_attention_balance(sixteenths, chunk)
        got = tw.gpu.decode_attention(0, q, v["block_table"][:6], v["seq_lens"][:6]).cpu().numpy().astype(np.float64)
        want = OA.paged_decode_attention(qx, tw.ora.k_pages[0], tw.ora.v_pages[0], tw.ora.block_table[:6], tw.ora.seq_lens[:6])
        err = np.abs(got - want)
        assert err.max() <= 1e-2 and err.mean() <= 1e-3, (sixteenths, chunk)
        tw.gpu.set_wait_limit_ns(0)                                                    # and run out again in between
        tw.gpu.decode_attention(0, q, v["block_table"][:6], v["seq_lens"][:6])
        torch.cuda.synchronize()
        assert tw.gpu.last_error()[1] & (1 << 6)
        tw.gpu.set_wait_limit_ns(2_000_000_000)
    got = tw.gpu.decode_attention(0, q, v["block_table"][:6], v["seq_lens"][:6]).cpu().numpy().astype(np.float64)
    want = OA.paged_decode_attention(qx, tw.ora.k_pages[0], tw.ora.v_pages[0], tw.ora.block_table[:6], tw.ora.seq_lens[:6])
    err = np.abs(got - want)
    assert err.max() <= 1e-2 and err.mean() <= 1e-3
    assert tw.status() == (0, 0)
