"""Random sequences of pool operations on the CUDA pool and the oracle pool side by side: after every operation the
free list, reference counts, block tables, lengths, live flags and status bits must be equal, bit for bit."""
import os

import numpy as np
import pytest
import torch

from oracle import attention as OA
from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W

from gpu_common import Twin, exact_f32, attention_errors

pytestmark = pytest.mark.gpu
N_SEEDS = int(os.environ.get("STEP_FUZZ_SEEDS", "12"))


def _dev(ids):
    return torch.tensor(list(ids), dtype=torch.int32, device="cuda:0")


@pytest.mark.parametrize("seed", range(N_SEEDS))
def test_random_operation_sequences(seed):
    g = np.random.default_rng(7000 + seed)
    payload = seed % 3 == 0                                    # every third seed also carries K/V and checks attention
    P = 16
    cfg = W.scaled(W.C1, n_traces=24, num_layers=2, num_q_heads=8, num_kv_heads=2, prefix_len=0, seed=7000 + seed)
    nb, max_pages, T = int(g.integers(40, 120)), int(g.integers(6, 14)), 24
    tw = Twin(cfg, nb, max_pages, T, shuffle=bool(seed & 1), store_payload=payload)
    o = tw.ora
    n_ops = 60 if payload else 140
    for step in range(n_ops):
        live = [t for t in range(T) if o.live[t]]
        op = g.choice(["fork", "append", "append", "append", "prune", "prune", "release", "finish"])
        if op == "fork" or not live:
            n = int(g.integers(1, 5))
            plen = int(g.choice([0, 5, 16, 37, 48]))
            full, rem = divmod(plen, P)
            if -(-plen // P) > max_pages or plen == 0 and payload:
                continue                                       # refused on the host, before anything is launched
            # a fork that cannot be served (too many traces in all, free list too short) is a no-op on both sides:
            # no ids, no blocks, a status bit
            ids, oids = tw.fork(n, plen)
            assert ids == oids                                 # (the status bits are compared below, after every operation)
        elif op == "append":
            k = int(g.integers(1, len(live) + 1))
            ids = [int(x) for x in g.choice(live, size=k, replace=False)]
            if g.random() < 0.15:
                dead = [t for t in range(T) if not o.live[t]]
                if dead:
                    ids.insert(int(g.integers(0, len(ids) + 1)), int(g.choice(dead)))     # flagged and skipped on both sides
            tw.append(ids, int(g.choice([1, 1, 2, 7, 16, 33])))
        elif op == "prune":
            scores = g.random(T).astype(np.float32)
            if g.random() < 0.3:
                scores[g.integers(0, T, size=3)] = scores[0]                                # ties
            if g.random() < 0.2:
                scores[g.integers(0, T)] = np.nan
            thr = float(g.choice([0.3, 0.6, 0.9, 1.0]))
            kf = float(g.choice([-1.0, 0.25, 0.5, 1.0]))
            pid, pn = tw.gpu.prune_if_saturated(torch.from_numpy(scores).cuda(), thr, kf)
            got = pid[:int(pn.item())].cpu().tolist()
            assert got == o.prune_if_saturated(scores, thr, kf), (step, got)
        elif op == "release":
            ids = [int(x) for x in g.choice(live, size=int(g.integers(1, min(4, len(live)) + 1)), replace=False)]
            tw.gpu.release_traces(_dev(ids))
            for t in ids:                                      # reclaimed in the order listed
                o.release_trace(t)
        else:
            ids = [int(x) for x in g.choice(live, size=int(g.integers(1, min(3, len(live)) + 1)), replace=False)]
            tw.gpu.finish_traces(_dev(ids), _dev(g.integers(0, 4, size=len(ids))))
            for t in ids:                                      # reclaimed in the order listed
                o.release_trace(t)
        try:
            tw.assert_meta_equal()
        except AssertionError as e:
            v = tw.gpu.views()
            fc = int(v["free_count"].item())
            raise AssertionError("step %d op %s ids %s: %s\n gpu free %s\n ora free %s" % (
                step, op, locals().get("ids"), e, v["free_list"][:fc].cpu().tolist(), o.free_list))
        mask, omask = tw.status()
        assert mask == omask, (step, op, mask, omask)
    if payload:
        n = o.next_trace
        if n:
            qb, qx = W.normal(cfg.seed, W.TID_Q, (n, 8, 128), "bf16")
            v = tw.gpu.views()
            for layer in (0, 1):
                got = exact_f32(tw.gpu.decode_attention(layer, H.to_device(qb, "bf16"), v["block_table"][:n], v["seq_lens"][:n]))
                want = OA.paged_decode_attention(qx, o.k_pages[layer], o.v_pages[layer], o.block_table[:n], o.seq_lens[:n])
                mx, mean = attention_errors(got, want)
                assert mx <= 1e-2 and mean <= 1e-3


@pytest.mark.parametrize("seed", range(N_SEEDS))
def test_random_scorer_launches(seed):
    """Random scorer widths, row counts, step-end densities and row-to-trace maps through score_steps (whichever
    first-layer kernel the library picks) against the oracle."""
    from test_gpu_parity import _scorer_case
    g = np.random.default_rng(9000 + seed)
    D = int(g.choice([64, 128, 320, 1000, 1024, 2560]))
    m = int(g.choice([8, 64, 96, 128, 192, 512]))
    T = int(g.integers(1, 70))
    M = int(g.choice([1, 7, 128, 129, 255, 300, 1000, 2500]))
    density = float(g.choice([0.0, 0.02, 0.3, 1.0]))
    rt = g.integers(0, T, size=M).astype(np.int32) if g.random() < 0.7 or M > T else None
    cfg = W.scaled(W.C1, n_traces=T, scorer_D=D, scorer_m=m, seed=9000 + seed)
    chunk = int(g.choice([0, 0, 200])) if M > 200 else 0
    _scorer_case(cfg, M, density, row_trace=rt, max_traces=T, max_score_rows=chunk or max(M, T),
                 mode=int(g.choice([0, 0, 1, -1])))


@pytest.mark.parametrize("seed", range(N_SEEDS))
def test_random_attention_launches(seed):
    """Random head groupings, trace counts, lengths (zeros and bare prompts included) and launch widths - so that the
    cuts between the warps' partitions of the KV stream fall everywhere - through decode_attention, its shared-prefix
    form and its allocation-free form, against the oracle."""
    g = np.random.default_rng(11000 + seed)
    hq, hkv = [(32, 8), (8, 8), (16, 2), (40, 8), (64, 8), (4, 1), (12, 4)][int(g.integers(0, 7))]
    n = int(g.integers(1, 40))
    prefix_len = int(g.choice([0, 9, 16, 50, 160]))
    cfg = W.scaled(W.C1, n_traces=n, num_layers=3, num_q_heads=hq, num_kv_heads=hkv, prefix_len=prefix_len, seed=11000 + seed)
    suffix = g.integers(0, int(g.choice([3, 40, 400])), size=n)
    if prefix_len == 0:
        suffix = np.maximum(suffix, 1)
    pages = int(sum(-(-(prefix_len + int(x)) // 16) for x in suffix)) + 8
    tw = Twin(cfg, pages, -(-(prefix_len + int(suffix.max())) // 16) + 2, n, shuffle=bool(seed & 1))
    ids, _ = tw.fork(n, prefix_len)
    for sel, inc in H.ragged_append_plan(np.asarray(suffix)):
        if inc > 0:
            assert all(tw.append([ids[i] for i in sel], inc))
    if n > 2 and g.random() < 0.5:                                     # a dead trace in the middle: length 0, table -1
        dead = int(g.integers(0, n))
        tw.gpu.release_traces(_dev([dead])); tw.ora.release_trace(dead)
    tw.gpu.set_attention_config(grid_ctas=int(g.integers(1, 149)))
    # how much of every sequence is handed out at run time, and in how small chunks (0 = equal shares only)
    tw.gpu.set_attention_balance(int(g.choice([0, 2, 4, 8, 12])), int(g.choice([1, 2, 5, 16])))
    o, v = tw.ora, tw.gpu.views()
    qb, qx = W.normal(cfg.seed, W.TID_Q, (n, hq, 128), "bf16")
    qd = H.to_device(qb, "bf16")
    want = OA.paged_decode_attention(qx, o.k_pages[0], o.v_pages[0], o.block_table[:n], o.seq_lens[:n])
    got = exact_f32(tw.gpu.decode_attention(0, qd, v["block_table"][:n], v["seq_lens"][:n]))
    mx, mean = attention_errors(got, want)
    assert mx <= 1e-2 and mean <= 1e-3, ("plain", mx, mean)
    # the three layers in one call (launches chained as programmatic dependents) = three plain calls, bit for bit
    q3 = torch.stack([qd, qd.flip(0), qd.roll(1, 0)]).contiguous()
    chained = tw.gpu.decode_attention_layers(0, q3, v["block_table"][:n], v["seq_lens"][:n])
    for l in range(3):
        assert torch.equal(chained[l], tw.gpu.decode_attention(l, q3[l], v["block_table"][:n], v["seq_lens"][:n])), ("layers", l)
    assert np.array_equal(exact_f32(chained[0]), got)
    if hq // hkv <= 8:
        out = torch.empty((n, hq, 128), dtype=torch.float32, device="cuda:0")
        tw.gpu.decode_attention_static(0, qd, v["block_table"][:n], v["seq_lens"][:n], out)
        mx, mean = attention_errors(exact_f32(out), want)
        assert mx <= 1e-2 and mean <= 1e-3, ("static", mx, mean)
    pp = prefix_len // 16
    live = [t for t in range(n) if o.live[t]]
    if pp and live:
        prefix = v["block_table"][live[0], :pp].contiguous()
        got = exact_f32(tw.gpu.decode_attention_shared_prefix(0, qd, v["block_table"][:n], v["seq_lens"][:n], prefix, pp))
        mx, mean = attention_errors(got, want)
        assert mx <= 1e-2 and mean <= 1e-3, ("shared", mx, mean)
    assert tw.status() == (0, 0)
