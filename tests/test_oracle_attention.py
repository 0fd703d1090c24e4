"""Pins for oracle/attention.py: nothing here re-uses the oracle's own formula."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import attention as A

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand(seed, *shape):
    return np.random.default_rng(seed).standard_normal(shape)


def test_closed_form_two_keys():
    # tests/golden/softmax_closed_form.txt: weights 1/4, 3/4
    with open(os.path.join(GOLD, "softmax_closed_form.txt")) as f:
        want = [float(x) for x in [l for l in f if l.startswith("o ")][0].split()[1:]]
    q = np.array([[2.0, 0, 0, 0]])
    K = np.zeros((2, 1, 4)); K[1, 0, 0] = math.log(3.0)
    V = np.zeros((2, 1, 4)); V[0, 0, 0] = 1.0; V[1, 0, 1] = 1.0
    np.testing.assert_allclose(A.dense_decode_attention(q, K, V)[0], want, atol=1e-15)


def test_single_position_returns_its_value():
    q, K, V = _rand(1, 4, 8), _rand(2, 1, 2, 8), _rand(3, 1, 2, 8)
    o = A.dense_decode_attention(q, K, V)
    for h in range(4):
        np.testing.assert_allclose(o[h], V[0, h // 2], atol=1e-15)


def test_identical_keys_give_mean_of_values():
    q = _rand(4, 2, 16)
    K = np.repeat(_rand(5, 1, 1, 16), 37, axis=0)
    V = _rand(6, 37, 1, 16)
    o = A.dense_decode_attention(q, K, V)
    np.testing.assert_allclose(o[0], V[:, 0].mean(axis=0), atol=1e-14)
    np.testing.assert_allclose(o[1], V[:, 0].mean(axis=0), atol=1e-14)


def test_dominant_logit_selects_its_value():
    d = 8
    q = np.zeros((1, d)); q[0, 0] = 1.0
    K = np.zeros((50, 1, d)); K[17, 0, 0] = 400.0      # logit 400/sqrt(8) >> 0
    V = _rand(7, 50, 1, d)
    np.testing.assert_allclose(A.dense_decode_attention(q, K, V)[0], V[17, 0], atol=1e-12)


def test_key_shift_invariance():
    q, K, V = _rand(8, 4, 16), _rand(9, 33, 2, 16), _rand(10, 33, 2, 16)
    u = _rand(11, 16)
    o1 = A.dense_decode_attention(q, K, V)
    o2 = A.dense_decode_attention(q, K + u, V)          # adds q.u/sqrt(d) to every logit
    np.testing.assert_allclose(o1, o2, atol=1e-12)


def test_output_inside_convex_hull_of_values():
    q, K, V = _rand(12, 4, 8), _rand(13, 40, 1, 8), _rand(14, 40, 1, 8)
    o = A.dense_decode_attention(q, K, V)
    assert np.all(o <= V[:, 0].max(axis=0) + 1e-12) and np.all(o >= V[:, 0].min(axis=0) - 1e-12)


def test_group_mapping_consecutive_heads_share_a_kv_head():
    # Hq = 4, Hkv = 2: heads 0,1 read kv head 0; heads 2,3 read kv head 1.
    d = 4
    q = np.tile(_rand(15, 1, d), (4, 1))                # the same query on every head
    K, V = _rand(16, 9, 2, d), _rand(17, 9, 2, d)
    o = A.dense_decode_attention(q, K, V)
    np.testing.assert_array_equal(o[0], o[1])
    np.testing.assert_array_equal(o[2], o[3])
    assert not np.allclose(o[1], o[2])
    # and head 1 equals a single-head problem on kv head 0 (h % G would pick kv head 1)
    o_single = A.dense_decode_attention(q[:1], K[:, :1], V[:, :1])
    np.testing.assert_allclose(o[1], o_single[0], atol=1e-15)


@pytest.mark.parametrize("Hq,Hkv,d,S", [(4, 1, 64, 97), (32, 8, 128, 300), (8, 8, 32, 5)])
def test_matches_library_sdpa(Hq, Hkv, d, S):
    # third opinion: torch's CPU scaled_dot_product_attention with K/V repeated G times
    q, K, V = _rand(20, Hq, d), _rand(21, S, Hkv, d), _rand(22, S, Hkv, d)
    G = Hq // Hkv
    tq = torch.from_numpy(q)[None, :, None, :]                                  # [1,Hq,1,d]
    tk = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(G, 0)[None]      # [1,Hq,S,d]
    tv = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0, :, 0, :].numpy()
    np.testing.assert_allclose(A.dense_decode_attention(q, K, V), want, atol=1e-12)


def _scatter_to_pages(Ks, Vs, P, num_blocks, perm):
    """Place contiguous per-trace K/V [S,Hkv,d] into pages; returns pages + table."""
    Hkv, d = Ks[0].shape[1:]
    kp = np.full((num_blocks, Hkv, P, d), np.nan)        # NaN poison: unused slots must not be read
    vp = np.full((num_blocks, Hkv, P, d), np.nan)
    max_pages = max(-(-len(K) // P) for K in Ks)
    bt = np.full((len(Ks), max_pages), -1, dtype=np.int64)
    nxt = 0
    for t, (K, V) in enumerate(zip(Ks, Vs)):
        for j in range(len(K)):
            if j % P == 0:
                bt[t, j // P] = perm[nxt]; nxt += 1
            b = bt[t, j // P]
            kp[b, :, j % P] = K[j]; vp[b, :, j % P] = V[j]
    return kp, vp, bt


def test_paged_equals_dense_on_unpaged_and_page_permutation_is_bit_invariant():
    rng = np.random.default_rng(30)
    lens = [1, 15, 16, 17, 64, 93, 0]
    Hq, Hkv, d, P = 4, 2, 16, 16
    Ks = [rng.standard_normal((S, Hkv, d)) for S in lens]
    Vs = [rng.standard_normal((S, Hkv, d)) for S in lens]
    q = rng.standard_normal((len(lens), Hq, d))
    nb = 64
    outs = []
    for perm in (np.arange(nb), rng.permutation(nb)):
        kp, vp, bt = _scatter_to_pages(Ks, Vs, P, nb, perm)
        outs.append(A.paged_decode_attention(q, kp, vp, bt, np.array(lens)))
    assert np.array_equal(outs[0], outs[1])               # same bits whatever the placement
    for t, S in enumerate(lens):
        np.testing.assert_array_equal(outs[0][t], A.dense_decode_attention(q[t], Ks[t], Vs[t]))
    assert np.all(outs[0][-1] == 0.0) and not np.isnan(outs[0]).any()


def test_split_evaluation_merges_to_direct():
    q, K, V = _rand(40, 1, 32), _rand(41, 200, 1, 32), _rand(42, 200, 1, 32)
    direct = A.dense_decode_attention(q, K, V)[0]
    cuts = [0, 7, 64, 65, 199, 200]
    parts = [A.partial_of_range(q[0], K[:, 0], V[:, 0], a, b) for a, b in zip(cuts[:-1], cuts[1:])]
    merged = A.merge_partials([p[0] for p in parts], [p[1] for p in parts], [p[2] for p in parts])
    np.testing.assert_allclose(merged, direct, atol=1e-13)


def test_large_logits_do_not_overflow():
    q = np.full((1, 4), 100.0)
    K = np.stack([np.full((1, 4), 50.0), np.full((1, 4), 49.0)])
    V = np.array([[[1.0, 0, 0, 0]], [[0, 1.0, 0, 0]]])
    o = A.dense_decode_attention(q, K, V)
    assert np.isfinite(o).all() and o[0, 0] > 0.999999


def test_flop_count():
    assert A.attention_flops(32, 128, 1000) == 4 * 32 * 128 * 1000


def test_shared_prefix_attention_definition():
    """With shared first pages it is the plain paged attention; with rows that do not share them it is dense attention
    over (shared pages ++ own positions) assembled by hand; short and empty rows give zeros."""
    g = np.random.default_rng(21)
    NB, Hkv, P, d, Hq = 20, 2, 4, 8, 4
    kp, vp = g.standard_normal((NB, Hkv, P, d)), g.standard_normal((NB, Hkv, P, d))
    q = g.standard_normal((4, Hq, d))
    shared = [7, 3]
    bt = np.full((4, 5), -1)
    bt[0, :4] = [7, 3, 10, 11]; bt[1, :3] = [7, 3, 12]; bt[2, :2] = [7, 3]; bt[3, :3] = [7, 3, 13]
    sl = np.array([14, 9, 8, 0])
    want = A.paged_decode_attention(q, kp, vp, bt, sl)
    got, short = A.paged_decode_attention_shared_prefix(q, kp, vp, bt, sl, shared)
    assert short == []
    np.testing.assert_array_equal(got, want)
    assert np.all(got[3] == 0)
    # rows whose own first pages differ: the shared blocks are used all the same
    bt2 = bt.copy(); bt2[0, :2] = [1, 2]; bt2[1, :2] = [-1, -1]
    got2, _ = A.paged_decode_attention_shared_prefix(q, kp, vp, bt2, sl, shared)
    np.testing.assert_array_equal(got2, want)
    # by hand for trace 0: 8 shared positions, then blocks 10 and 11 (6 of their 8 slots)
    K = np.concatenate([kp[7].swapaxes(0, 1), kp[3].swapaxes(0, 1), kp[10].swapaxes(0, 1), kp[11].swapaxes(0, 1)[:2]])
    V = np.concatenate([vp[7].swapaxes(0, 1), vp[3].swapaxes(0, 1), vp[10].swapaxes(0, 1), vp[11].swapaxes(0, 1)[:2]])
    np.testing.assert_allclose(got[0], A.dense_decode_attention(q[0], K, V), rtol=0, atol=1e-15)
    # a row shorter than the prefix
    sl3 = np.array([14, 5, 8, 0])
    got3, short3 = A.paged_decode_attention_shared_prefix(q, kp, vp, bt, sl3, shared)
    assert short3 == [1] and np.all(got3[1] == 0)
    np.testing.assert_array_equal(got3[0], want[0])
    # split identity: prefix partial merged with the suffix partial is the whole
    Kg, Vg = K[:, 0], V[:, 0]
    parts = [A.partial_of_range(q[0, 1], Kg, Vg, 0, 8), A.partial_of_range(q[0, 1], Kg, Vg, 8, 14)]
    np.testing.assert_allclose(A.merge_partials(*zip(*parts)), got[0, 1], rtol=0, atol=1e-14)
