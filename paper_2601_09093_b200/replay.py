"""Replay of what a serving engine WITHOUT pruning does when the KV pool fills (Sec. 2 "Latency Bottleneck"; Table 3's
"wait" row): it preempts the trace admitted last, frees its KV, keeps it in a waiting queue, and when a finishing trace
makes room reconstructs the waiting trace's whole KV before it decodes again.  Host-side scheduling only: every pool
operation goes through the `ops` object, so the same schedule can drive the CUDA pool (bench.py) or any other pool
with the same five operations (the tests).  No attention or scoring arithmetic lives here.

ops: free() -> free blocks now; fork_all(n, prompt_len) -> ids; fork_one(seq_len) -> id (a trace whose first seq_len
positions are written at once: the reconstruction); append(ids) (one token each); release(ids); finish(ids);
step(ids) (optional: whatever the caller runs per decode iteration, e.g. attention)."""
from __future__ import annotations

import collections


def preempt_and_recompute(ops, final_len, prompt_len, page, max_iterations=10 ** 7):
    """Runs len(final_len) traces from a shared prompt to their final lengths.  Returns the schedule's counters:
    iterations, decode_steps (tokens generated), preemptions, recomputed_tokens, waiting_trace_iterations (the sum over
    iterations of the queue length: the paper's waiting time in units of decode iterations), max_waiting."""
    n = len(final_len)
    ids = list(ops.fork_all(n, prompt_len))
    S = [prompt_len] * n
    running = list(range(n))                              # admission order
    waiting = collections.deque()
    c = dict(iterations=0, decode_steps=0, preemptions=0, recomputed_tokens=0, waiting_trace_iterations=0, max_waiting=0)
    while (running or waiting) and c["iterations"] < max_iterations:
        # room for this iteration's tokens: preempt from the back of the admission order until the new pages fit
        need = sum(1 for t in running if S[t] % page == 0)
        free = ops.free()
        while need > free and len(running) > 1:
            t = running.pop()
            ops.release([ids[t]])
            waiting.appendleft(t)
            c["preemptions"] += 1
            free = ops.free()
            need = sum(1 for u in running if S[u] % page == 0)
        if running:
            cur = [ids[t] for t in running]
            ops.append(cur)
            for t in running:
                S[t] += 1
            c["decode_steps"] += len(running)
            if hasattr(ops, "step"):
                ops.step(cur)
            done = [t for t in running if S[t] >= final_len[t]]
            if done:
                ops.finish([ids[t] for t in done])
                running = [t for t in running if S[t] < final_len[t]]
        # re-admit from the front of the queue while a reconstructed trace (and its next token) fits
        while waiting:
            t = waiting[0]
            pages = -(-S[t] // page) + (1 if S[t] % page == 0 else 0)
            if pages > ops.free() - sum(1 for u in running if S[u] % page == 0):
                break
            waiting.popleft()
            ids[t] = ops.fork_one(S[t])
            running.append(t)
            c["recomputed_tokens"] += S[t]
        c["iterations"] += 1
        c["waiting_trace_iterations"] += len(waiting)
        c["max_waiting"] = max(c["max_waiting"], len(waiting))
    c["unfinished"] = len(running) + len(waiting)
    return c
