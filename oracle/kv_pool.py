"""Oracle: paged KV pool bookkeeping, memory trigger and prune (Algorithm 1).

TEST INFRASTRUCTURE ONLY - never imported by the product path.

What the paper fixes
--------------------
* InitTraces(P, N): N traces start from one prompt (Algorithm 1, first line).
* Trigger (Sec. 3.2): prune when GPU memory is full and the KV cache for the
  next decoding step cannot be scheduled.
* Rule (Sec. 3.2, Algorithm 1): evict the trace with the lowest average step
  score, release its KV cache at once, drop it from the trace set.

What the paper leaves open, and the reading taken here
------------------------------------------------------
* "Memory full" as an integer predicate on a block pool:
      used  = total - free_count
      need  = #{live t : S_t % P == 0}      (blocks the next step must pop)
      limit = floor(threshold * total)      (threshold widened to float64)
      saturated  <=>  used + need > limit
  threshold = 1 is the paper's sentence word for word; a fraction below 1 is
  the "maximum GPU memory utilisation" knob of the sensitivity study.
* How many to evict per trigger: the paper evicts exactly one (the argmin);
  keep_frac < 0 selects that.  keep_frac in (0, 1] is a generalisation: keep
  n_keep = max(1, ceil(keep_frac * n_live - 1e-6)) best traces, evict the rest.
* Ties: the lower trace id ranks higher (is kept).  NaN ranks below everything.
* Score of a trace with no scored step: supplied by the caller (see scorer.py).
* Shared prompt pages are reference counted; a block returns to the free list
  when its count reaches zero.
* Orders (so that the free list is reproducible bit for bit):
  - the free list is a stack; allocation pops from the end, release pushes
    to the end; it starts as [total-1, ..., 1, 0] so the first pop is block 0;
  - fork: shared full pages pop in page order, then (only if the prompt length
    is not a multiple of P) one private tail block per trace in trace order;
  - append: traces in the order given, pages in ascending order;
  - reclaim: evicted traces in ascending id, pages in ascending order.

Error conditions never raise: they set a bit in `status` and skip the affected
trace, mirroring a device that must not trap.
"""
from __future__ import annotations

import math

import numpy as np

OK, ERR_INVALID_ARG, ERR_NO_BLOCKS, ERR_BAD_TRACE, ERR_CAPACITY = 0, 1, 2, 3, 4


class KVPoolOracle:
    def __init__(self, num_layers, num_kv_heads, head_dim, page_size, num_blocks,
                 max_traces, max_pages_per_trace, store_payload=True):
        self.L, self.Hkv, self.d, self.P = num_layers, num_kv_heads, head_dim, page_size
        self.num_blocks, self.max_traces, self.max_pages = num_blocks, max_traces, max_pages_per_trace
        self.block_table = np.full((max_traces, max_pages_per_trace), -1, dtype=np.int64)
        self.seq_lens = np.zeros(max_traces, dtype=np.int64)
        self.live = np.zeros(max_traces, dtype=bool)
        self.refcount = np.zeros(num_blocks, dtype=np.int64)
        self.free_list = list(range(num_blocks - 1, -1, -1))
        self.next_trace = 0
        self.status = 0
        self.store_payload = store_payload
        if store_payload:
            shape = (num_layers, num_blocks, num_kv_heads, page_size, head_dim)
            self.k_pages = np.zeros(shape, dtype=np.float64)
            self.v_pages = np.zeros(shape, dtype=np.float64)

    # ------------------------------------------------------------------ helpers
    @property
    def free_count(self):
        return len(self.free_list)

    @property
    def used(self):
        return self.num_blocks - len(self.free_list)

    def _flag(self, code):
        self.status |= 1 << code

    def _pop(self):
        return self.free_list.pop()

    def _write_row(self, t, pos, k_row, v_row):
        """k_row, v_row : [L, Hkv, d] for logical position pos of trace t."""
        if not self.store_payload:
            return
        b = int(self.block_table[t, pos // self.P])
        s = pos % self.P
        self.k_pages[:, b, :, s, :] = k_row
        self.v_pages[:, b, :, s, :] = v_row

    # --------------------------------------------------------------- InitTraces
    def fork_prefix(self, n_traces, prefix_len, k_prefix=None, v_prefix=None):
        """Start n_traces traces that share one prompt of prefix_len tokens.

        k_prefix, v_prefix : [L, Hkv, prefix_len, d] (ignored without payload).
        Returns the list of new trace ids, or [] with a status bit set.
        """
        P = self.P
        if n_traces < 1 or prefix_len < 0:
            self._flag(ERR_INVALID_ARG)
            return []
        if self.next_trace + n_traces > self.max_traces or math.ceil(prefix_len / P) > self.max_pages:
            self._flag(ERR_CAPACITY)
            return []
        full, rem = divmod(prefix_len, P)
        if full + (n_traces if rem else 0) > self.free_count:
            self._flag(ERR_NO_BLOCKS)
            return []
        ids = list(range(self.next_trace, self.next_trace + n_traces))
        self.next_trace += n_traces
        shared = [self._pop() for _ in range(full)]
        for b in shared:
            self.refcount[b] = n_traces
        for t in ids:
            self.block_table[t, :full] = shared
            if rem:
                b = self._pop()
                self.refcount[b] = 1
                self.block_table[t, full] = b
            self.seq_lens[t] = prefix_len
            self.live[t] = True
        if self.store_payload and prefix_len:
            for t in ids:
                for pos in range(prefix_len):
                    self._write_row(t, pos, k_prefix[:, :, pos, :], v_prefix[:, :, pos, :])
        return ids

    # ---------------------------------------------------------------- append_kv
    def append_kv(self, trace_ids, n_tokens, k_new=None, v_new=None):
        """Append n_tokens positions to each listed trace.

        k_new, v_new : [n, n_tokens, L, Hkv, d].  Returns per-trace success flags.
        """
        P = self.P
        ok = []
        for i, t in enumerate(trace_ids):
            t = int(t)
            if t < 0 or t >= self.max_traces or not self.live[t]:
                self._flag(ERR_BAD_TRACE)
                ok.append(False)
                continue
            S = int(self.seq_lens[t])
            have = -(-S // P)
            want = -(-(S + n_tokens) // P)
            if want > self.max_pages:
                self._flag(ERR_CAPACITY)
                ok.append(False)
                continue
            if want - have > self.free_count:
                self._flag(ERR_NO_BLOCKS)
                ok.append(False)
                continue
            for page in range(have, want):
                b = self._pop()
                self.refcount[b] = 1
                self.block_table[t, page] = b
            if self.store_payload:
                for j in range(n_tokens):
                    self._write_row(t, S + j, k_new[i, j], v_new[i, j])
            self.seq_lens[t] = S + n_tokens
            ok.append(True)
        return ok

    # -------------------------------------------------------------------- prune
    def saturated(self, threshold) -> bool:
        need = int(np.sum(self.live & (self.seq_lens % self.P == 0)))
        limit = math.floor(float(np.float32(threshold)) * self.num_blocks)
        return self.used + need > limit

    @staticmethod
    def rank_order(scores, live_ids):
        """Live ids from best to worst: score descending, id ascending, NaN last."""
        def key(t):
            s = float(np.float32(scores[t]))
            if math.isnan(s):
                return (1, 0.0, t)
            return (0, -s, t)
        return sorted(live_ids, key=key)

    def n_keep(self, keep_frac, n_live):
        if keep_frac < 0:
            return n_live - 1                     # the paper's rule: evict the argmin only
        return max(1, math.ceil(float(np.float32(keep_frac)) * n_live - 1e-6))

    def prune_if_saturated(self, scores, threshold, keep_frac, on_evict=None):
        """Returns the evicted trace ids in ascending order ([] if nothing fired)."""
        if not self.saturated(threshold):
            return []
        live_ids = [t for t in range(self.max_traces) if self.live[t]]
        if not live_ids:
            return []
        keep = self.n_keep(keep_frac, len(live_ids))
        order = self.rank_order(scores, live_ids)
        evicted = sorted(order[keep:]) if keep < len(live_ids) else []
        for t in evicted:
            self.release_trace(t)
            if on_evict is not None:
                on_evict(t)
        return evicted

    def release_trace(self, t):
        """ReleaseKVCache(t): give back the trace's pages, clear its state."""
        n_pages = -(-int(self.seq_lens[t]) // self.P)
        for page in range(n_pages):
            b = int(self.block_table[t, page])
            self.refcount[b] -= 1
            if self.refcount[b] == 0:
                self.free_list.append(b)
        self.block_table[t, :] = -1
        self.seq_lens[t] = 0
        self.live[t] = False

    # --------------------------------------------------------------- invariants
    def check_invariants(self):
        """Raises AssertionError when the bookkeeping is inconsistent."""
        fl = self.free_list
        assert len(set(fl)) == len(fl), "duplicate block on the free list"
        counts = np.zeros(self.num_blocks, dtype=np.int64)
        for t in range(self.max_traces):
            n_pages = -(-int(self.seq_lens[t]) // self.P)
            if not self.live[t]:
                assert self.seq_lens[t] == 0 and np.all(self.block_table[t] == -1)
                continue
            row = self.block_table[t, :n_pages]
            assert np.all(row >= 0) and np.all(row < self.num_blocks)
            assert len(set(row.tolist())) == n_pages, "a trace maps one block twice"
            assert np.all(self.block_table[t, n_pages:] == -1)
            counts[row] += 1
        assert np.array_equal(counts, self.refcount), "refcount != number of referencing traces"
        in_use = set(np.nonzero(counts)[0].tolist())
        assert in_use.isdisjoint(fl), "a referenced block is on the free list"
        assert len(in_use) + len(fl) == self.num_blocks, "used + free != total"

    def bytes_per_token(self, elem_bytes):
        return self.L * self.Hkv * self.d * 2 * elem_bytes


def weighted_vote(answers, weights):
    """Weighted majority vote (Algorithm 1, last line; Sec. 3.3).

    answers : answer id per surviving trace; weights : its final trace score.
    The answer with the largest summed weight wins; ties go to the smaller id.
    """
    totals = {}
    for a, w in zip(answers, weights):
        totals[int(a)] = totals.get(int(a), 0.0) + float(w)
    if not totals:
        return None
    best = max(totals.values())
    return min(a for a, w in totals.items() if w == best)
