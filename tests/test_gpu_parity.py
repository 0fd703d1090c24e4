"""GPU parity: every call of the C ABI against the CPU oracle on the same seeded inputs."""
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

# tolerances for bf16-in / fp32-accumulate attention (max and mean absolute error) and for scores (absolute)
ATT_MAX, ATT_MEAN, SCORE_TOL = 1e-2, 1e-3, 1e-3


def _oracle_attention(tw: Twin, layer, q_exact, n):
    o = tw.ora
    return OA.paged_decode_attention(q_exact, o.k_pages[layer], o.v_pages[layer], o.block_table[:n], o.seq_lens[:n])


def _gpu_attention(tw: Twin, layer, q_dev, n):
    v = tw.gpu.views()
    return tw.gpu.decode_attention(layer, q_dev, v["block_table"][:n], v["seq_lens"][:n])


def _build(cfg, suffix, num_blocks=None, shuffle=False, extra_pages=2):
    P = cfg.page_size
    n = len(suffix)
    pages = int(sum(-(-(cfg.prefix_len + s) // P) for s in suffix)) + 8
    tw = Twin(cfg, num_blocks or pages, max(-(-(cfg.prefix_len + int(max(suffix))) // P) + extra_pages, 4), n, shuffle=shuffle)
    ids, oids = tw.fork(n, cfg.prefix_len)
    assert ids == oids
    for sel, inc in H.ragged_append_plan(np.asarray(suffix)):
        assert all(tw.append([ids[i] for i in sel], inc))
    return tw, ids


def _check_attention(tw, cfg, n, layers=(0,), max_tol=ATT_MAX, mean_tol=ATT_MEAN):
    for layer in layers:
        qb, qx = W.normal(cfg.seed, W.TID_Q, (n, cfg.num_q_heads, cfg.head_dim), cfg.dtype, sub=layer)
        got = exact_f32(_gpu_attention(tw, layer, H.to_device(qb, cfg.dtype), n))
        want = _oracle_attention(tw, layer, qx, n)
        mx, mean = attention_errors(got, want)
        assert mx <= max_tol and mean <= mean_tol, (layer, mx, mean)
    assert tw.status() == (0, 0)


# ------------------------------------------------------------------ pool
def test_c0_pool_metadata_and_payload_roundtrip():
    cfg = W.C0
    suffix = W.suffix_lengths(cfg)
    tw, ids = _build(cfg, suffix, num_blocks=cfg.num_blocks)
    tw.assert_meta_equal()
    v = tw.gpu.views()
    for t in (0, 3, 7):
        S = int(tw.ora.seq_lens[t])
        k, vv = tw.gpu.read_kv(0, 0, v["block_table"][t], S)
        K, V = OA.gather_trace_kv(tw.ora.k_pages[0], tw.ora.v_pages[0], tw.ora.block_table[t], S)
        np.testing.assert_array_equal(exact_f32(k), K[:, 0])
        np.testing.assert_array_equal(exact_f32(vv), V[:, 0])
    assert tw.status() == (0, 0)


def test_fork_with_partial_page_and_token_by_token_append():
    cfg = W.scaled(W.C0, prefix_len=37, num_layers=2, num_kv_heads=2, num_q_heads=4)
    tw = Twin(cfg, 64, 12, 3)
    ids, oids = tw.fork(3, 37)
    assert ids == oids == [0, 1, 2]
    tw.assert_meta_equal()
    for step in range(30):
        tw.append(ids, 1)
    tw.append(ids[:2], 21)
    tw.assert_meta_equal()
    _check_attention(tw, cfg, 3, layers=(0, 1), max_tol=1e-4, mean_tol=1e-5)


def test_bf16_swizzled_layout_roundtrip_multi_layer():
    cfg = W.scaled(W.C1, n_traces=3, num_layers=3, prefix_len=40)
    tw, ids = _build(cfg, [5, 70, 33])
    tw.assert_meta_equal()
    v = tw.gpu.views()
    for layer in range(3):
        for head in (0, 5, 7):
            for t in range(3):
                S = int(tw.ora.seq_lens[t])
                k, vv = tw.gpu.read_kv(layer, head, v["block_table"][t], S)
                K, V = OA.gather_trace_kv(tw.ora.k_pages[layer], tw.ora.v_pages[layer], tw.ora.block_table[t], S)
                np.testing.assert_array_equal(exact_f32(k), K[:, head])
                np.testing.assert_array_equal(exact_f32(vv), V[:, head])


def test_error_conditions_are_flagged_not_fatal():
    cfg = W.scaled(W.C0, prefix_len=16)
    tw = Twin(cfg, 3, 2, 3, store_payload=False)
    ids, _ = tw.fork(2, 16)
    assert tw.append([0, 1, 5], 16) == [True, True, False]
    assert tw.status() == (1 << 3, 1 << 3)
    assert tw.append([0], 1) == [False]
    assert tw.status() == (1 << 4, 1 << 4)
    tw.assert_meta_equal()
    tw2 = Twin(cfg, 2, 4, 2, store_payload=False)
    tw2.fork(2, 16)
    assert tw2.append([0, 1], 16) == [True, False]
    assert tw2.status() == (1 << 2, 1 << 2)
    tw2.assert_meta_equal()
    # a fork the free list cannot serve is a no-op
    tw3 = Twin(cfg, 1, 4, 2, store_payload=False)
    tw3.gpu.fork_prefix(2, 32, torch.zeros((1, 1, 32, 64), device="cuda"), torch.zeros((1, 1, 32, 64), device="cuda"))
    assert tw3.gpu.last_error()[1] == 1 << 2 and tw3.gpu.stats() == dict(used=0, free=1, total=1, live_traces=0)


def test_a_fork_that_fails_consumes_no_ids_and_can_be_retried():
    """Row i of the loop's inputs is trace i, so ids must not be lost to a fork the pool could not serve: the retry
    after blocks were freed gets the ids the failed fork would have got - as in the oracle."""
    cfg = W.scaled(W.C0, prefix_len=0)
    tw = Twin(cfg, 6, 4, 4, store_payload=False)
    ids, oids = tw.fork(2, 40)                                   # 2 shared pages + a private partial page each: 4 blocks
    assert ids == oids == [0, 1]
    ids, oids = tw.fork(2, 40)                                   # needs 4 more, 2 are free
    assert ids == oids == []
    assert tw.status() == (1 << 2, 1 << 2)
    tw.assert_meta_equal()
    tw.gpu.release_traces(torch.tensor([0, 1], dtype=torch.int32, device="cuda"))
    tw.ora.release_trace(0); tw.ora.release_trace(1)
    ids, oids = tw.fork(2, 40)                                   # now it fits, and takes ids 2 and 3 on both sides
    assert ids == oids == [2, 3]
    assert tw.append(ids, 8) == [True, True]
    tw.assert_meta_equal()
    ids, oids = tw.fork(1, 16)                                   # a fifth trace in a pool of four
    assert ids == oids == []
    assert tw.status() == (1 << 4, 1 << 4)
    tw.assert_meta_equal()
    tw.gpu.reset(); torch.cuda.synchronize()
    assert tw.gpu.fork_prefix(1, 0, None, None) == [0]           # a reset pool starts again at id 0


def test_an_id_listed_twice_is_served_once_and_flagged():
    """append_kv, kv_pool_release_traces and kv_pool_finish_traces take lists of distinct ids; a repeat is flagged
    (BAD_TRACE) and skipped, so the pool ends as if the list had named the trace once at its first place."""
    cfg = W.scaled(W.C0, prefix_len=32)
    tw = Twin(cfg, 64, 8, 6, store_payload=False)
    ids, _ = tw.fork(6, 32)
    dev = lambda x: torch.tensor(x, dtype=torch.int32, device="cuda")
    z = torch.zeros((6, 20, 1, 1, 64), device="cuda")
    tw.gpu.append_kv(dev([3, 1, 3, 5, 1, 0]), 20, z, z)           # (a list may not be longer than max_traces)
    assert tw.ora.append_kv([3, 1, 5, 0], 20) == [True] * 4
    tw.assert_meta_equal()
    assert tw.gpu.last_error()[1] == 1 << 3
    tw.gpu.release_traces(dev([4, 1, 4, 1]))
    tw.ora.release_trace(4); tw.ora.release_trace(1)
    tw.assert_meta_equal()
    assert tw.gpu.last_error()[1] == 1 << 3
    tw.gpu.finish_traces(dev([5, 0, 5]), dev([7, 8, 9]))
    tw.ora.release_trace(5); tw.ora.release_trace(0)
    tw.assert_meta_equal()
    assert tw.gpu.last_error()[1] == 1 << 3
    vv = tw.gpu.vote_views()
    assert vv["answer"][5].item() == 7 and vv["answer"][0].item() == 8
    assert tw.gpu.stats()["live_traces"] == 2                    # traces 2 and 3; the shared prompt pages are still theirs
    tw.gpu.release_traces(dev([2, 3, 2]))
    tw.ora.release_trace(2); tw.ora.release_trace(3)
    tw.assert_meta_equal()
    assert tw.gpu.stats()["used"] == 0


def test_host_side_argument_checks():
    pool = H.make_pool(W.C0, 8, 4)
    z = torch.zeros(4, device="cuda")
    with pytest.raises(B.StepError):
        pool.prune_if_saturated(None, 0.95, 0.0)
    with pytest.raises(B.StepError):
        pool.prune_if_saturated(None, 1.5, 0.5)
    with pytest.raises(B.StepError):
        pool.decode_attention(3, z, z, z)
    with pytest.raises(B.StepError):
        B.kv_pool_required_bytes(num_layers=1, num_q_heads=3, num_kv_heads=2, head_dim=64, page_size=16,
                                 num_blocks=4, max_traces=1, max_pages_per_trace=1, dtype=0)


# ------------------------------------------------------------------ attention
def test_c0_attention_fp32():
    cfg = W.C0
    tw, ids = _build(cfg, W.suffix_lengths(cfg), num_blocks=cfg.num_blocks)
    _check_attention(tw, cfg, cfg.n_traces, max_tol=1e-4, mean_tol=1e-5)


@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (64, 8), (8, 8), (16, 1), (24, 2), (40, 10)])
def test_bf16_attention_ragged_small(Hq, Hkv):
    # several pages per warp partition, partial last pages, a one-token and an empty trace
    cfg = W.scaled(W.C1, n_traces=9, num_q_heads=Hq, num_kv_heads=Hkv, prefix_len=48)
    suffix = [0, 1, 15, 16, 17, 700, 2049, 333, 5000]
    tw, ids = _build(cfg, suffix)
    _check_attention(tw, cfg, 9)
    # same inputs through the scalar kernel
    tw.gpu.set_attention_config(fast_path=-1)
    _check_attention(tw, cfg, 9)


def test_bf16_attention_empty_and_single_token_traces():
    cfg = W.scaled(W.C1, n_traces=4, prefix_len=0)
    tw = Twin(cfg, 16, 4, 4)
    ids, _ = tw.fork(4, 0)
    tw.append([1], 1)
    tw.append([3], 20)
    _check_attention(tw, cfg, 4)
    v = tw.gpu.views()
    qb, qx = W.normal(cfg.seed, W.TID_Q, (4, 32, 128), "bf16")
    out = exact_f32(_gpu_attention(tw, 0, H.to_device(qb, "bf16"), 4))
    assert np.all(out[0] == 0) and np.all(out[2] == 0)
    k, vv = tw.gpu.read_kv(0, 2, v["block_table"][1], 1)
    np.testing.assert_allclose(out[1, 8:12], np.tile(exact_f32(vv), (4, 1)), atol=1e-6)   # S = 1: o = V[0]


def test_attention_grid_sizes_and_page_shuffle_agree():
    # page-permutation invariance on the GPU, and independence from how the KV stream is partitioned
    cfg = W.scaled(W.C1, n_traces=6, prefix_len=64)
    suffix = [100, 900, 2500, 31, 1200, 64]
    outs = []
    for shuffle in (False, True):
        tw, ids = _build(cfg, suffix, num_blocks=512, shuffle=shuffle)
        qb, qx = W.normal(cfg.seed, W.TID_Q, (6, 32, 128), "bf16")
        qd = H.to_device(qb, "bf16")
        want = _oracle_attention(tw, 0, qx, 6)
        for grid in (0, 1, 3, 37, 500):
            tw.gpu.set_attention_config(grid_ctas=grid)
            got = exact_f32(_gpu_attention(tw, 0, qd, 6))
            mx, mean = attention_errors(got, want)
            assert mx <= ATT_MAX and mean <= ATT_MEAN, (shuffle, grid, mx, mean)
            outs.append(got)
        assert tw.status() == (0, 0)
    assert np.abs(outs[0] - outs[5]).max() < 1e-5      # only the physical placement differs


@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (16, 1)])
def test_attention_is_the_same_however_the_pages_are_handed_out(Hq, Hkv):
    """Equal shares only, the default, and up to three quarters of every sequence in chunks of one page and more
    (hundreds of chunks, fetched by whichever warp is free): every setting within tolerance of the oracle, a
    setting's repeat bit-identical, and the shared-prefix call under the same settings too."""
    cfg = W.scaled(W.C1, n_traces=9, num_q_heads=Hq, num_kv_heads=Hkv, prefix_len=96)
    suffix = [0, 1, 15, 16, 17, 700, 2049, 333, 5000]
    tw, ids = _build(cfg, suffix)
    qb, qx = W.normal(cfg.seed, W.TID_Q, (9, Hq, 128), "bf16")
    qd = H.to_device(qb, "bf16")
    want = _oracle_attention(tw, 0, qx, 9)
    v = tw.gpu.views()
    pp = 96 // 16
    prefix_blocks = v["block_table"][0, :pp].clone()
    with pytest.raises(Exception):
        tw.gpu.set_attention_balance(13)
    for grid in (0, 5):
        tw.gpu.set_attention_config(grid_ctas=grid)
        for sixteenths, chunk in [(0, 0), (4, 16), (4, 1), (12, 1), (12, 3), (8, 64)]:
            tw.gpu.set_attention_balance(sixteenths, chunk)
            got = exact_f32(_gpu_attention(tw, 0, qd, 9))
            mx, mean = attention_errors(got, want)
            assert mx <= ATT_MAX and mean <= ATT_MEAN, (grid, sixteenths, chunk, mx, mean)
            again = exact_f32(_gpu_attention(tw, 0, qd, 9))
            assert np.array_equal(got, again), (grid, sixteenths, chunk)
            out = tw.gpu.decode_attention_shared_prefix(0, qd, v["block_table"][:9], v["seq_lens"][:9], prefix_blocks, pp)
            mx, mean = attention_errors(exact_f32(out), want)
            assert mx <= ATT_MAX and mean <= ATT_MEAN, ("shared prefix", grid, sixteenths, chunk, mx, mean)
    assert tw.status() == (0, 0)


def test_attention_padding_slots_do_not_leak():
    # unused slots of the last page hold NaN bit patterns: the result must not see them
    cfg = W.scaled(W.C1, n_traces=2, prefix_len=0)
    tw = Twin(cfg, 8, 4, 2)
    tw.gpu.kv_storage.view(torch.int16).fill_(0x7FC0)   # bf16 NaN everywhere
    tw.fork(2, 0)
    tw.append([0, 1], 5)
    tw.append([1], 13)
    _check_attention(tw, cfg, 2)


@pytest.mark.parametrize("scale", [24.0, 1.0 / 64])
def test_attention_with_peaked_and_flat_softmax(scale):
    """Queries 24x larger make the softmax a near-argmax (logits of several hundred: only the max subtraction keeps
    exp in range); queries 64x smaller make it a near-mean.  Both through the tensor-core and the scalar kernel."""
    cfg = W.scaled(W.C1, n_traces=5, prefix_len=48, seed=515)
    tw, ids = _build(cfg, [0, 7, 300, 1500, 64])
    qb, qx = W.normal(cfg.seed, W.TID_Q, (5, 32, 128), "bf16", std=scale)
    want = _oracle_attention(tw, 0, qx, 5)
    for fast in (1, -1):
        tw.gpu.set_attention_config(fast_path=fast)
        got = exact_f32(_gpu_attention(tw, 0, H.to_device(qb, "bf16"), 5))
        assert np.isfinite(got).all()
        mx, mean = attention_errors(got, want)
        assert mx <= ATT_MAX and mean <= ATT_MEAN, (scale, fast, mx, mean)
    assert tw.status() == (0, 0)


def test_bad_block_table_is_flagged():
    cfg = W.scaled(W.C1, n_traces=1, prefix_len=32)
    tw, ids = _build(cfg, [40])
    v = tw.gpu.views()
    bt = v["block_table"][:1].clone()
    bt[0, 1] = 10 ** 6
    q = torch.zeros((1, 32, 128), dtype=torch.bfloat16, device="cuda")
    tw.gpu.decode_attention(0, q, bt, v["seq_lens"][:1])
    assert tw.gpu.last_error()[1] == 1 << 7


# ------------------------------------------------------------------ scorer
def _scorer_case(cfg, M, density, row_trace=None, bias=0.05, max_traces=None, max_score_rows=0, mode=0,
                 tc_min_rows=0, expect_tc=None, sample=0):
    """score_steps against the oracle.  mode / tc_min_rows pick the first-layer kernel (0 = the library's
    own choice); expect_tc checks which one ran (hidden units per CTA of the tensor-core kernel, 0 = the
    CUDA-core kernel).  sample > 0: only that many boundary rows (spread over the list, ends included) are
    given to the oracle - for launches too large for it; the running means are then checked against the
    GPU's own step scores only."""
    T = max_traces or cfg.n_traces
    pool = H.make_pool(cfg, 8, 4, T, max_score_rows=max_score_rows)
    pool.set_scorer_config(mode, tc_min_rows)
    (W1b, W1x), (b1b, b1x), (w2b, w2x), b2 = W.scorer_weights(cfg, bias_std=bias)
    wts = B.ScorerWeights(H.to_device(W1b, cfg.dtype), H.to_device(b1b, cfg.dtype), H.to_device(w2b, cfg.dtype), b2,
                          H.step_dtype(cfg))
    hb, hx = W.normal(cfg.seed, W.TID_HID, (M, cfg.scorer_D), cfg.dtype)
    mask = W.boundary_mask(cfg, M, density=density)
    rt_dev = None if row_trace is None else torch.from_numpy(row_trace.astype(np.int32)).cuda()
    got = pool.score_steps(H.to_device(hb, cfg.dtype), torch.from_numpy(mask).cuda(), rt_dev, wts)
    if expect_tc is not None:
        info = pool.score_launch_info()
        assert info["tc_units"] == expect_tc, info
    g = got.cpu().numpy()
    assert np.isnan(g[mask == 0]).all()
    assert not np.isnan(g[mask == 1]).any()
    if sample:
        rows = np.flatnonzero(mask)
        pick = rows[np.unique(np.linspace(0, len(rows) - 1, sample).astype(np.int64))]
        W1d, b1d, w2d = W1x.astype(np.float64), b1x.astype(np.float64), w2x.astype(np.float64)
        want_s = np.array([OS.step_score(hx[i], W1d, b1d, w2d, b2) for i in pick])
        assert np.abs(g[pick] - want_s).max() <= SCORE_TOL
        want = None
    else:
        want = OS.score_steps(hx, mask, W1x, b1x, w2x, b2)
        if mask.any():
            assert np.abs(g[mask == 1] - want[mask == 1]).max() <= SCORE_TOL
    ts = OS.TraceScores(T)
    ts.update(g, mask, row_trace)                       # running means from the GPU's own step scores
    v = pool.views()
    np.testing.assert_allclose(v["trace_scores"].cpu().numpy(), ts.scores(), atol=2e-6 if M <= 3000 else 1e-5)
    np.testing.assert_array_equal(v["score_cnt"].cpu().numpy(), ts.cnt)
    if want is not None:
        ts2 = OS.TraceScores(T)
        ts2.update(want, mask, row_trace)               # and within tolerance of the all-oracle means
        assert np.abs(v["trace_scores"].cpu().numpy() - ts2.scores()).max() <= SCORE_TOL
    assert pool.last_error() == (0, 0)
    return pool, wts, g, mask


def test_c0_scorer_fp32():
    _scorer_case(W.C0, 8, 1.0, bias=0.0)


# mode -1: the CUDA-core first layer; mode 0: the library's choice (for at most 256 candidate rows: the one-launch kernel)
@pytest.mark.parametrize("mode", [-1, 0])
def test_scorer_bf16_decode_shape(mode):
    _scorer_case(W.C1, 64, 1.0 / 8, mode=mode, expect_tc=0)


@pytest.mark.parametrize("mode", [-1, 0])
def test_scorer_bf16_all_and_none_boundaries(mode):
    _scorer_case(W.C1, 64, 1.0, mode=mode)
    _scorer_case(W.C1, 64, 0.0, mode=mode, expect_tc=0)


@pytest.mark.parametrize("mode", [-1, 0])
def test_scorer_batched_rows_with_row_trace_and_chunking(mode):
    cfg = W.C1
    M = 64 * 40 + 13
    rt = (np.arange(M) % 64).astype(np.int32)
    _scorer_case(cfg, M, 1.0 / 16, row_trace=rt, max_score_rows=M, mode=mode)
    _scorer_case(cfg, M, 1.0 / 16, row_trace=rt, max_score_rows=1000, mode=mode)    # several launches


def test_scorer_c4_shape_cuda_cores():
    _scorer_case(W.C4, 128, 0.1, mode=-1, expect_tc=0)


def test_scorer_odd_shapes_take_the_cuda_core_kernel():
    """D not a multiple of 64 / m not a multiple of 64: outside the tensor-core kernel's shapes."""
    _scorer_case(W.scaled(W.C1, scorer_D=1000, scorer_m=96), 64, 0.5, mode=0, expect_tc=0)
    _scorer_case(W.scaled(W.C1, scorer_D=1024, scorer_m=96), 64, 0.5, mode=1, expect_tc=0)


# ---- the tensor-core first layer (tcgen05): same rows, same tolerance
def test_scorer_tensor_core_partial_tile():
    """Fewer rows than one 128-row tile, forced onto the tensor cores (narrowest slices)."""
    _scorer_case(W.C1, 64, 1.0 / 8, mode=1, expect_tc=64)
    _scorer_case(W.C1, 64, 1.0, mode=1, expect_tc=64)
    _scorer_case(W.C1, 64, 0.0, mode=1, expect_tc=0)              # no boundary row: nothing to do


def test_scorer_tensor_core_c4_shape():
    """m = 1024, D = 5120: sixteen 64-unit slices, 80 k-chunks."""
    _scorer_case(W.C4, 128, 0.5, mode=1, expect_tc=64)


def test_scorer_tensor_core_ragged_tiles_with_row_trace():
    """Several tiles and a ragged last one, rows scattered over the input by the mask, many rows per trace."""
    cfg = W.C1
    M = 64 * 40 + 13
    rt = (np.arange(M) % 64).astype(np.int32)
    _scorer_case(cfg, M, 1.0 / 4, row_trace=rt, max_score_rows=M, expect_tc=64)       # ~640 rows
    _scorer_case(cfg, M, 1.0 / 16, row_trace=rt, max_score_rows=M, tc_min_rows=100, expect_tc=64)


@pytest.mark.parametrize("M", [300, 64 * 40 + 13])
def test_scorer_tensor_core_every_row_listed_ragged(M):
    """Every candidate row ends a step, so the tensor-core kernel fetches the rows as tiles of the caller's array
    instead of gathering them: a second row half that lies partly (or wholly) past the end of the array, several
    tiles, and a call cut into launches of 1000 rows (each launch sees its own part of the array)."""
    rt = (np.arange(M) % 64).astype(np.int32)
    _scorer_case(W.C1, M, 1.0, row_trace=rt, max_score_rows=M, mode=1)
    _scorer_case(W.C1, M, 1.0, row_trace=rt, max_score_rows=1000, mode=1)


def test_scorer_picks_the_cuda_core_kernel_below_the_row_threshold():
    rt = (np.arange(512) % 64).astype(np.int32)
    _scorer_case(W.C1, 512, 1.0 / 8, row_trace=rt, max_score_rows=512, tc_min_rows=128, expect_tc=0)   # ~64 rows
    _scorer_case(W.C1, 512, 1.0, row_trace=rt, max_score_rows=512, mode=-1, expect_tc=0)    # forced off


@pytest.mark.parametrize("rows,units", [(4800, 128), (9600, 256), (19000, 256)])
def test_scorer_tensor_core_wide_slices_sampled(rows, units):
    """Launches large enough that the device picks 128- and 256-unit slices (several items per CTA, both
    accumulators in use).  The oracle scores a sample of rows; the CUDA-core kernel, itself checked against
    the oracle above, cross-checks every row."""
    cfg = W.C1
    rt = (np.arange(rows) % 64).astype(np.int32)
    _, _, g_tc, mask = _scorer_case(cfg, rows, 1.0, row_trace=rt, max_score_rows=rows, expect_tc=units, sample=96)
    _, _, g_cc, _ = _scorer_case(cfg, rows, 1.0, row_trace=rt, max_score_rows=rows, mode=-1, expect_tc=0, sample=8)
    assert np.abs(g_tc - g_cc).max() <= 1e-4


def test_scorer_running_mean_accumulates_across_calls():
    cfg = W.C1
    pool, wts, g1, m1 = _scorer_case(cfg, 64, 0.5)
    hb, hx = W.normal(cfg.seed, W.TID_HID, (64, cfg.scorer_D), cfg.dtype, sub=7)
    mask = W.boundary_mask(cfg, 64, sub=7, density=0.5)
    g2 = pool.score_steps(H.to_device(hb, cfg.dtype), torch.from_numpy(mask).cuda(), None, wts).cpu().numpy()
    ts = OS.TraceScores(64)
    ts.update(g1, m1); ts.update(g2, mask)
    np.testing.assert_allclose(pool.views()["trace_scores"].cpu().numpy(), ts.scores(), atol=1e-6)


# ------------------------------------------------------------------ step-end detection from sampled tokens
def _vocab_case(seed, vocab_size, M, density):
    from oracle import steps as OSt
    vocab = W.synthetic_vocab(seed, vocab_size, step_end_frac=0.02)
    table = B.step_end_table_from_vocab(vocab)
    ends = np.flatnonzero(table.numpy())
    ids = W.token_ids(seed, M, vocab_size, ends, density)
    return vocab, table.cuda(), ids, OSt.step_end_mask(ids, vocab)


def test_detect_step_ends_matches_the_oracle_bit_for_bit():
    pool = H.make_pool(W.C0, 8, 4, 8)
    for M in (1, 255, 4097, 70001):
        vocab, table, ids, want = _vocab_case(5, 32000, M, 1.0 / 64)
        got = pool.detect_step_ends(torch.from_numpy(ids).cuda(), table).cpu().numpy()
        np.testing.assert_array_equal(got, want)
    assert pool.last_error() == (0, 0)
    ids[3], ids[9] = -7, 32000                                   # ids outside the vocabulary end no step, and are flagged
    got = pool.detect_step_ends(torch.from_numpy(ids).cuda(), table).cpu().numpy()
    assert got[3] == 0 and got[9] == 0
    assert pool.last_error()[1] == 1 << 1


@pytest.mark.parametrize("mode", [-1, 0])
def test_score_steps_tokens_equals_score_steps_on_the_oracle_mask(mode):
    cfg = W.C1
    M = 64 * 30 + 5
    vocab, table, ids, mask = _vocab_case(cfg.seed, 32000, M, 1.0 / 16)
    rt = (np.arange(M) % 64).astype(np.int32)
    pool_a, wts, g_mask, _ = _scorer_case(cfg, M, 0.0, row_trace=rt, max_score_rows=1000, mode=mode)   # builds pool + weights
    hb, hx = W.normal(cfg.seed, W.TID_HID, (M, cfg.scorer_D), cfg.dtype)
    hid = H.to_device(hb, cfg.dtype)
    rt_dev = torch.from_numpy(rt).cuda()
    ref = pool_a.score_steps(hid, torch.from_numpy(mask).cuda(), rt_dev, wts).cpu().numpy()
    ref_scores = pool_a.views()["trace_scores"].cpu().numpy().copy()
    pool_b = H.make_pool(cfg, 8, 4, 64, max_score_rows=1000)
    pool_b.set_scorer_config(mode, 0)
    mask_out = torch.empty(M, dtype=torch.uint8, device="cuda")
    got = pool_b.score_steps_tokens(hid, torch.from_numpy(ids).cuda(), table, rt_dev, wts, boundary_mask_out=mask_out).cpu().numpy()
    np.testing.assert_array_equal(mask_out.cpu().numpy(), mask)
    np.testing.assert_array_equal(got, ref)                     # same kernels, same rows: identical bits (NaN where no step ends)
    np.testing.assert_array_equal(pool_b.views()["trace_scores"].cpu().numpy(), ref_scores)
    want = OS.score_steps(hx, mask, *[x for x in _exact_weights(cfg)])
    assert np.abs(got[mask == 1] - want[mask == 1]).max() <= SCORE_TOL
    assert pool_b.last_error() == (0, 0)


def _exact_weights(cfg):
    (_, W1x), (_, b1x), (_, w2x), b2 = W.scorer_weights(cfg, bias_std=0.05)
    return W1x, b1x, w2x, b2


@pytest.mark.parametrize("mode", [-1, 1])
def test_scorer_saturating_logits(mode):
    """Weights twenty times larger than usual drive the logit to tens or hundreds: the sigmoid must saturate to 0 / 1
    without overflow or NaN, on the CUDA-core and on the tensor-core first layer."""
    cfg = W.scaled(W.C1, n_traces=16, scorer_D=512, scorer_m=128, seed=616)
    pool = H.make_pool(cfg, 8, 4, 16, max_score_rows=300)
    pool.set_scorer_config(mode, 0)
    (W1b, W1x), (b1b, b1x), (w2b, w2x), b2 = W.scorer_weights(cfg, std=1.0, bias_std=0.5)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16"), H.to_device(b1b, "bf16"), H.to_device(w2b, "bf16"), b2, B.STEP_BF16)
    hb, hx = W.normal(cfg.seed, W.TID_HID, (300, 512), "bf16")
    mask = np.ones(300, dtype=np.uint8)
    rt = (np.arange(300) % 16).astype(np.int32)
    got = pool.score_steps(H.to_device(hb, "bf16"), torch.from_numpy(mask).cuda(), torch.from_numpy(rt).cuda(), wts).cpu().numpy()
    want = OS.score_steps(hx, mask, W1x, b1x, w2x, b2)
    assert np.isfinite(got).all() and got.min() >= 0.0 and got.max() <= 1.0
    assert (got == 0.0).any() or (got == 1.0).any() or (np.minimum(got, 1 - got).min() < 1e-6)      # it does saturate
    assert np.abs(got - want).max() <= SCORE_TOL
    assert pool.last_error() == (0, 0)


@pytest.mark.parametrize("hq,hkv", [(32, 8), (32, 2)])
def test_attention_layers_call_equals_layer_by_layer_calls(hq, hkv):
    """decode_attention_layers (every launch after the first a programmatic dependent of the one before) gives, bit
    for bit, what one decode_attention call per layer gives, and both agree with the oracle."""
    cfg = W.scaled(W.C1, n_traces=9, num_layers=5, num_q_heads=hq, num_kv_heads=hkv, prefix_len=40, seed=717)
    tw, ids = _build(cfg, [0, 300, 17, 1200, 64, 5, 900, 33, 2000])
    tw.gpu.release_traces(torch.tensor([4], dtype=torch.int32, device="cuda")); tw.ora.release_trace(4)
    qb, qx = W.normal(cfg.seed, W.TID_Q, (5, 9, hq, 128), "bf16")
    qd = H.to_device(qb, "bf16")
    v = tw.gpu.views()
    for grid in (148, 5):
        tw.gpu.set_attention_config(grid_ctas=grid)
        for layer0, nl in ((0, 5), (2, 3), (4, 1)):
            got = tw.gpu.decode_attention_layers(layer0, qd[:nl], v["block_table"][:9], v["seq_lens"][:9])
            for l in range(nl):
                one = tw.gpu.decode_attention(layer0 + l, qd[l], v["block_table"][:9], v["seq_lens"][:9])
                assert torch.equal(got[l], one), (grid, layer0, l)
                want = _oracle_attention(tw, layer0 + l, qx[l], 9)
                mx, mean = attention_errors(exact_f32(got[l]), want)
                assert mx <= ATT_MAX and mean <= ATT_MEAN
    # many short launches in a row: every launch's partials and tickets share one scratch area
    big = torch.stack([tw.gpu.decode_attention_layers(0, qd, v["block_table"][:9], v["seq_lens"][:9]).clone() for _ in range(20)])
    assert all(torch.equal(big[0], b) for b in big[1:])
    assert tw.status() == (0, 0)
    with pytest.raises(B.StepError):
        tw.gpu.decode_attention_layers(3, qd[:3], v["block_table"][:9], v["seq_lens"][:9])     # layers 3, 4, 5: one too many


@pytest.mark.parametrize("grid", [148, 5])
def test_dependent_launch_waits_for_the_kernel_that_writes_q(grid):
    """decode_attention_dependent is scheduled while the kernel before it - here a 256 MB copy whose first rows are
    the queries - is still running, and must not read q before that kernel has completed: the buffer holds NaN bit
    patterns until the copy lands.  Results equal the plain call's, bit for bit, layer after layer."""
    cfg = W.scaled(W.C1, n_traces=9, num_layers=3, prefix_len=40, seed=818)
    tw, ids = _build(cfg, [0, 300, 17, 1200, 64, 5, 900, 33, 2000])
    qb, qx = W.normal(cfg.seed, W.TID_Q, (3, 9, 32, 128), "bf16")
    qd = H.to_device(qb, "bf16")
    v = tw.gpu.views()
    tw.gpu.set_attention_config(grid_ctas=grid)
    n_q = 9 * 32 * 128
    big_src = torch.zeros(128 << 20, dtype=torch.bfloat16, device="cuda")
    big_dst = torch.empty_like(big_src)
    for rep in range(3):
        for l in range(3):
            big_dst.view(torch.int16).fill_(0x7FC0)              # NaN everywhere, the query rows included
            big_src[:n_q] = qd[l].reshape(-1)
            torch.mul(big_src, 1, out=big_dst)                   # the kernel that "produces" q (an elementwise kernel, not a memcpy)
            got = tw.gpu.decode_attention_dependent(l, big_dst[:n_q].view(9, 32, 128), v["block_table"][:9], v["seq_lens"][:9])
            one = tw.gpu.decode_attention(l, qd[l], v["block_table"][:9], v["seq_lens"][:9])
            assert torch.equal(got, one), (rep, l)
    want = _oracle_attention(tw, 2, qx[2], 9)
    mx, mean = attention_errors(exact_f32(got), want)
    assert mx <= ATT_MAX and mean <= ATT_MEAN
    assert tw.status() == (0, 0)
    # a pool the tensor-core kernel does not cover takes the ordinary launch
    tw0, _ = _build(W.C0, [5, 40])
    q0b, q0x = W.normal(W.C0.seed, W.TID_Q, (2, 4, 64), "fp32")
    v0 = tw0.gpu.views()
    a = tw0.gpu.decode_attention_dependent(0, H.to_device(q0b, "fp32"), v0["block_table"][:2], v0["seq_lens"][:2])
    b = tw0.gpu.decode_attention(0, H.to_device(q0b, "fp32"), v0["block_table"][:2], v0["seq_lens"][:2])
    assert torch.equal(a, b)


def test_read_stream_probe_runs_clean_both_ways():
    buf = torch.empty((64 << 20) + 4096, dtype=torch.uint8, device="cuda")      # not a whole number of 8 KiB pieces
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    for chained in (0, 1):
        B.read_stream_probe(buf, 5, chained, err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    with pytest.raises(B.StepError):
        B.read_stream_probe(buf[:4096], 1, 0, err)
