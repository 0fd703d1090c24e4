"""Oracle: Algorithm 1 (the STEP loop) on the oracle's pool, scorer and step-end test.

TEST INFRASTRUCTURE ONLY - never imported by the product path.

Algorithm 1, in the paper's order and names:

    T <- InitTraces(P, N)
    while T != {}:
        for each trace t in T:
            (x, h) <- NextToken(t)
            if "\\n\\n" in x:   y <- f(h);  update score_t with y
            if GPUMemoryFull:  t* <- argmin score_t;  ReleaseKVCache(t*);  T <- T \\ {t*}
    answer <- WeightedVote(T, {score_t})

and Sec. 3.3: "once all traces have either completed or been pruned" the vote uses the final trace scores.

NextToken is the model's forward pass, which is not part of the method's hot path here: its results (the
sampled token x, the hidden state h, the new K/V rows) are inputs.  Readings where the paper is silent:

* One pass of the for-each loop is taken as a batch: all live traces receive their token, then the trigger
  is tested once (the engine the paper builds on also decodes all running traces in one step).
* A trace completes when it samples the end-of-sequence token.  Its score_t at that moment is its final
  score; its KV is released at once; it leaves T but takes part in the vote.  Evicted traces do not vote.
* The trigger / eviction rule is the pool oracle's (kv_pool.py): threshold 1.0 with keep_frac < 0 is the
  paper's rule word for word.
* With the one-eviction rule a single eviction may not free enough blocks when many traces reach a page
  boundary in the same iteration; `max_evictions` lets the trigger be tested, and the rule applied, that many
  times in a row (each test sees the pool the last eviction left).  1 is the pseudo-code as printed.
* Order within an iteration: cache write (append) -> step-end test and scorer -> completions (ascending
  trace id) -> trigger and eviction.
"""
from __future__ import annotations

import numpy as np

from . import attention as OA
from . import scorer as OS
from . import steps as OSt
from .kv_pool import KVPoolOracle, weighted_vote


class Algorithm1Oracle:
    def __init__(self, pool: KVPoolOracle, n_traces, W1, b1, w2, b2, vocab_texts, eos_token, threshold, keep_frac,
                 unscored_score=1.0, max_evictions=1):
        self.pool, self.n = pool, n_traces
        self.W1, self.b1, self.w2, self.b2 = W1, b1, w2, b2
        self.vocab, self.eos = vocab_texts, int(eos_token)
        self.threshold, self.keep_frac = threshold, keep_frac
        self.ts = OS.TraceScores(pool.max_traces, unscored_score)
        self.finished = {}                 # trace id -> (final score, answer)
        self.n_evicted = 0
        self.max_evictions = max(1, int(max_evictions))

    def live(self):
        return [t for t in range(self.n) if self.pool.live[t]]

    def iteration(self, token_ids, hidden, answers=None, k_new=None, v_new=None, rank_scores=None, step_scores=None,
                  q=None):
        """One pass of the while loop.  Row i of every input is trace i.

        rank_scores : if given, the trace scores the eviction ranks by (a test passes the device's float32
                      scores here so that both sides take the decision on the same numbers);
        step_scores : if given, the step scores folded into score_t instead of this oracle's own (same reason).
        q           : [layers, n, Hq, d]; if given (and the pool stores K/V), NextToken's attention of those layers
                      over each live trace's cache, new token included, is returned too.
        Returns what happened: step-end mask of the live rows, the oracle's own step scores, completed and
        evicted trace ids."""
        live = self.live()
        if live:
            kn = None if k_new is None else np.asarray(k_new)[live]
            vn = None if v_new is None else np.asarray(v_new)[live]
            self.pool.append_kv(live, 1, kn, vn)
        att = None
        if q is not None:
            p, n = self.pool, len(token_ids)
            att = np.stack([OA.paged_decode_attention(q[l], p.k_pages[l], p.v_pages[l], p.block_table[:n], p.seq_lens[:n])
                            for l in range(len(q))])
        mask = OSt.step_end_mask(token_ids, self.vocab)
        is_live = np.zeros(len(token_ids), dtype=bool)
        is_live[live] = True
        mask = (mask.astype(bool) & is_live).astype(np.uint8)
        ys = OS.score_steps(hidden, mask, self.W1, self.b1, self.w2, self.b2)
        self.ts.update(ys if step_scores is None else step_scores, mask)
        done = [t for t in live if int(token_ids[t]) == self.eos]
        for t in done:
            self.finished[t] = (self.ts.score(t), -1 if answers is None else int(answers[t]))
            self.pool.release_trace(t)
            self.ts.clear(t)
        scores = self.ts.scores() if rank_scores is None else rank_scores
        evicted = []
        for _ in range(self.max_evictions):
            if rank_scores is None:
                scores = self.ts.scores()
            gone = self.pool.prune_if_saturated(scores, self.threshold, self.keep_frac, on_evict=self.ts.clear)
            if not gone:
                break
            evicted += gone
        self.n_evicted += len(evicted)
        return dict(mask=mask, step_scores=ys, finished=done, evicted=evicted, attention=att)

    def vote(self, final_scores=None):
        """WeightedVote over the completed traces; final_scores (by trace id) overrides the recorded scores."""
        ids = sorted(t for t, (_, a) in self.finished.items() if a >= 0)
        w = [self.finished[t][0] if final_scores is None else float(final_scores[t]) for t in ids]
        return weighted_vote([self.finished[t][1] for t in ids], w)

    def run(self, token_ids, hidden, answers, max_iterations=None):
        """token_ids [iterations, n], hidden [iterations, n, D].  Runs until T is empty; returns (answer, log)."""
        log = []
        for i in range(len(token_ids) if max_iterations is None else max_iterations):
            if not self.live():
                break
            log.append(self.iteration(token_ids[i], hidden[i], answers))
        return self.vote(), log
