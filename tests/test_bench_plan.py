"""Host logic of bench.py (no GPU): the sizes it plans for each workload hold what the run will put into them."""
import math
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2601_09093_b200 import workloads as W  # noqa: E402


@pytest.mark.parametrize("traces,threshold", [(0, 0.0), (16, 0.0), (32, 0.5), (32, 0.9)])
def test_memory_saturated_plan_stays_below_the_trigger_during_the_timed_steps(traces, threshold):
    steps_total = bench.planned_steps(10, 3, 10)                    # as run_ours counts them
    cfg, suffix, nb, max_pages, layers = bench.workload_plan("c3", 0, steps_total, None, traces, threshold)
    T, P = cfg.n_traces, cfg.page_size
    assert T == (traces or 64) and layers == 36 and nb == 65536
    limit = math.floor(float(np.float32(cfg.threshold)) * nb)
    shared = cfg.prefix_len // P
    # after every planned step: blocks in use plus the blocks the next step needs must not exceed the limit
    final = cfg.prefix_len + int(suffix[0]) + steps_total
    used = shared + T * (-(-final // P) - shared)
    assert used + T <= limit
    # and the pool is nearly full: one more page per trace beyond the margin would cross it
    assert used + T * (steps_total // P + 4) > limit
    # the block table has room for the prune cycles (4 survivors sharing the pool at the end)
    assert max_pages >= shared + (limit - shared) // 4
    assert cfg.bytes_per_token == 147456


@pytest.mark.parametrize("name", ["c1", "c2", "c4"])
def test_fixed_trace_set_plans_hold_every_page(name):
    steps_total = 40
    cfg, suffix, nb, max_pages, layers = bench.workload_plan(name, 0, steps_total)
    P = cfg.page_size
    pages = cfg.prefix_len // P + sum(-(-(int(s) + steps_total) // P) for s in suffix)
    assert pages + cfg.n_traces <= math.floor(float(np.float32(cfg.threshold)) * nb)     # the trigger stays quiet
    assert max_pages * P >= cfg.prefix_len + int(suffix.max()) + steps_total
    assert len(suffix) == cfg.n_traces and suffix.min() >= cfg.suffix_lo and suffix.max() <= cfg.suffix_hi


def test_ragged_append_plan_gives_every_trace_its_length():
    from paper_2601_09093_b200 import harness as H
    lengths = np.array([5, 0, 17, 5, 300, 1])
    got = np.zeros(len(lengths), dtype=np.int64)
    for sel, inc in H.ragged_append_plan(lengths):
        assert inc > 0 and list(sel) == sorted(sel)
        got[sel] += inc
    assert np.array_equal(got, lengths)


def test_scorer_shapes_are_the_papers_model_widths():
    got = {name: (bench.scorer_shape(name).scorer_D, bench.scorer_shape(name).scorer_m) for name in ("c1", "c4", "d2560", "d5120")}
    assert got == {"c1": (4096, 512), "c4": (5120, 1024), "d2560": (2560, 512), "d5120": (5120, 512)}
