#!/usr/bin/env python
"""Benchmark of the STEP decode hot path (libstep) on B200.

A "step" is one decode iteration of Algorithm 1 for all live traces on device-resident state:
append_kv (one new token per trace, all layers) -> decode_attention for every layer ->
score_steps on the step-end hidden states -> prune_if_saturated.

Default workload: the 64-trace memory-saturated configuration (Qwen3-8B KV layout, 36 layers,
8 KV heads, d = 128, bf16, page 16, pool of ~150 GB) in the state just below the 95 % trigger,
i.e. the headline state of the prune benchmark.  Inputs are synthetic and seeded.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "paged decode-attn KV GB/s (fraction of B200 HBM peak); trace-decode-steps/sec"
UNIT = "trace-decode-steps/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c3", "c1", "c2", "c4", "scorer", "prefix", "replay", "append"])
    ap.add_argument("--prefix-len", type=int, default=8192, help="prefix workload: tokens of the shared prompt")
    ap.add_argument("--suffix-max", type=int, default=512, help="prefix workload: traces hold 1 .. this many tokens of their own")
    ap.add_argument("--scorer-rows", type=int, default=65536, help="rows of the batched scorer workload")
    ap.add_argument("--scorer-density", type=float, default=1.0, help="fraction of those rows that end a step")
    ap.add_argument("--scorer-shape", default="c1", choices=["c1", "c4", "d2560", "d5120"],
                    help="scorer workload: D 4096 / m 512 (c1), D 5120 / m 1024 (c4), or the paper's other model widths with m 512")
    ap.add_argument("--traces", type=int, default=0, help="c3 only: sampling budget N (traces sharing the pool); 0 = 64")
    ap.add_argument("--threshold", type=float, default=0.0, help="c3 only: pool fraction at which the trigger fires; 0 = 0.95")
    ap.add_argument("--no-aux", action="store_true", help="skip the scorer / prune-cycle measurements after the timed steps")
    ap.add_argument("--num-blocks", type=int, default=0, help="override the pool size (blocks)")
    ap.add_argument("--grid", type=int, default=0, help="CTAs of the attention launch (0 = library default)")
    ap.add_argument("--balance", type=int, default=-1,
                    help="sixteenths of every sequence's pages that the attention launches of the timed steps hand out at run "
                         "time (kv_pool_set_attention_balance); -1 = 2 when a step chains several layers' launches, else the library's 4")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def attention_dram_traffic_ratio():
    """DRAM bytes moved per algorithmic byte by attn_mma_kernel, from the counters of one ncu capture kept in
    profiles/attn_mma_kernel_dram_traffic.txt (dram__bytes_read.sum + dram__bytes_write.sum against the launch's
    algorithmic bytes).  The kernel streams every page once, so traffic grows in proportion to the algorithmic bytes
    and the larger workloads scale this figure.  The file names the kernel sources it was taken from by their
    SHA-256; if they have changed since, the counters no longer describe the kernel and None is returned."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "attn_mma_kernel_dram_traffic.txt")
    if not os.path.exists(path):
        return None, "no counters on file"
    kv = {}
    with open(path) as f:
        for line in f:
            if "=" in line and not line.lstrip().startswith("#"):
                k, val = line.split("=", 1)
                kv[k.strip()] = val.strip()
    h = hashlib.sha256()
    for name in ("attention.cu", "async_copy.cuh"):
        with open(os.path.join(ROOT, "paper_2601_09093_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    if kv.get("kernel_sources_sha256") != h.hexdigest():
        return None, "the kernel changed since the counters in %s were taken" % os.path.relpath(path, ROOT)
    ratio = (float(kv["dram_bytes_read"]) + float(kv["dram_bytes_write"])) / float(kv["algorithmic_bytes"])
    return ratio, os.path.relpath(path, ROOT) + ": ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch on the one-layer 64-trace workload, scaled by algorithmic bytes"


def measured_peaks(key="hbm_gbs", fallback=6650.0):
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        if key in d:
            return float(d[key]), "measured"
    return fallback, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thr = threading.Thread(target=self._read, daemon=True)
            self.thr.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except Exception:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
def workload_plan(name, num_blocks_override, steps_total, free_bytes=None, traces=0, threshold=0.0):
    """Shapes of the benchmark state: config, per-trace suffix lengths, pool size."""
    from paper_2601_09093_b200 import workloads as W
    if name == "c3":
        cfg = W.C3
        if traces or threshold:
            # the paper's sweeps: sampling budget N = 16 / 32 / 64 and the KV memory budget 0.5 - 0.9
            cfg = W.scaled(cfg, n_traces=traces or cfg.n_traces, threshold=threshold or cfg.threshold,
                           name="%s-N%d-thr%.2f" % (cfg.name, traces or cfg.n_traces, threshold or cfg.threshold))
        nb = num_blocks_override or cfg.num_blocks
        block_bytes = cfg.bytes_per_token * cfg.page_size
        if free_bytes is not None:
            fit = int((free_bytes - (6 << 30)) // block_bytes)
            nb = min(nb, fit)
        limit = math.floor(float(np.float32(cfg.threshold)) * nb)
        shared = cfg.prefix_len // cfg.page_size
        margin_pages = -(-steps_total // cfg.page_size) + 1
        p0 = (limit - shared) // cfg.n_traces - margin_pages         # private pages per trace at the start
        if p0 < 1:
            raise SystemExit("pool too small for the memory-saturated workload")
        suffix = np.full(cfg.n_traces, p0 * cfg.page_size, dtype=np.int64)
        # the prune cycles that follow the timed steps grow the survivors until 2 traces share the pool
        max_pages = max(shared + p0 + margin_pages + 2, shared + limit // 4 + 64)
        return cfg, suffix, nb, max_pages, cfg.num_layers
    cfg = {"c1": W.C1, "c2": W.C2, "c4": W.C4}[name]
    suffix = W.suffix_lengths(cfg)
    shared = cfg.prefix_len // cfg.page_size
    pages = shared + int(sum(-(-(s + steps_total) // cfg.page_size) + 1 for s in suffix))
    # these workloads time attention at a fixed trace set: size the pool so the trigger stays quiet
    nb = num_blocks_override or int(pages / float(np.float32(cfg.threshold)) * 1.02) + 64
    max_pages = -(-(cfg.prefix_len + int(suffix.max()) + steps_total) // cfg.page_size) + 2
    phys_layers = cfg.num_layers
    if free_bytes is not None:
        per_layer = nb * cfg.bytes_per_token_layer * cfg.page_size
        phys_layers = max(1, min(cfg.num_layers, int((free_bytes - (6 << 30)) // per_layer)))
    return cfg, suffix, nb, max_pages, phys_layers


def planned_steps(K, Wm, e2e_steps):
    """Tokens every trace gains over a whole default run (timed steps, the per-layer-call legs, the end-to-end leg, the
    library-driven loop): the state is sized so that the trigger stays quiet through all of them."""
    return Wm + K + 3 * (2 + K) + (Wm + e2e_steps) + 4 + ALG1_ITERATIONS_ONE_LAYER + 3 + ALG1_GRAPH_ITERATIONS + 2


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2601_09093_b200 import binding as B, harness as H, ranks as R, workloads as W
    from paper_2601_09093_b200 import build as _build

    rank, local_rank, world = R.rank_env()
    if rank == 0:
        _build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    B.lib()

    K, Wm = args.steps, max(args.warmup, 3)
    e2e_steps = 0 if args.no_e2e else K
    steps_total = planned_steps(K, Wm, e2e_steps)
    free_b, total_b = torch.cuda.mem_get_info(dev)
    cfg, suffix, nb, max_pages, phys_layers = workload_plan(args.workload, args.num_blocks, steps_total, free_b,
                                                            args.traces, args.threshold)
    cfg_pool = W.scaled(cfg, num_layers=phys_layers)
    T, L = cfg.n_traces, cfg.num_layers
    pool = H.make_pool(cfg_pool, nb, max_pages, T, max_score_rows=T, device=dev)
    if args.grid:
        pool.set_attention_config(grid_ctas=args.grid)
    # In a chain of launches (decode_attention_layers) an SM that is done early starts on the next layer, so less of
    # the stream needs handing out at run time than for a launch on its own: measured on one device, 36-layer steps
    # took 21.29 / 20.59 / 20.76 / 20.85 ms with 0 / 2 / 4 / 6 sixteenths, one-layer steps 0.489 / 0.464 / 0.451 / 0.456 ms.
    LIB_BALANCE = 4
    step_balance = args.balance if args.balance >= 0 else (2 if L > 1 else LIB_BALANCE)
    pool.set_attention_balance(step_balance)
    if cfg.shuffle_pages:
        H.shuffle_free_list(pool, cfg.seed + rank)
    t_fill = time.time()
    append_log = []                                    # every append_kv call, for the oracle's replay of the prune cycles
    ids = H.fill_random_device(pool, cfg_pool, suffix, seed=cfg.seed + 7919 * rank,
                               chunk_tokens=max(16, (1 << 28) // (T * cfg_pool.bytes_per_token)), log=append_log)
    torch.cuda.synchronize()
    t_fill = time.time() - t_fill
    v = pool.views()
    ids_dev = torch.tensor(ids, dtype=torch.int32, device=dev)

    # rotating sets of per-step inputs (device copies and pinned host copies of the same values)
    gen = torch.Generator(device=dev); gen.manual_seed(cfg.seed + 1 + rank)
    NSETS = 2
    def rnd(*shape):
        return torch.randn(shape, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    sets = []
    mask_np = [W.boundary_mask(cfg, T, sub=100 + i) for i in range(NSETS)]
    for i, mk in enumerate(mask_np):
        if not mk.any():
            mk[i % T] = 1                # every timed step scores at least one step end (the expected number per step is one or two)
    for i in range(NSETS):
        s = dict(q=rnd(L, T, cfg.num_q_heads, cfg.head_dim), k=rnd(T, 1, phys_layers, cfg.num_kv_heads, cfg.head_dim),
                 v=rnd(T, 1, phys_layers, cfg.num_kv_heads, cfg.head_dim), h=rnd(T, cfg.scorer_D),
                 m=torch.from_numpy(mask_np[i]).to(dev))
        s["host"] = {k: s[k].cpu().pin_memory() for k in ("q", "k", "v", "h", "m")}
        sets.append(s)
    (W1b, _), (b1b, _), (w2b, _), b2 = W.scorer_weights(cfg)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16", dev), H.to_device(b1b, "bf16", dev), H.to_device(w2b, "bf16", dev), b2, B.STEP_BF16)
    out = torch.empty((L, T, cfg.num_q_heads, cfg.head_dim), dtype=torch.float32, device=dev)
    step_scores = torch.empty(T, dtype=torch.float32, device=dev)
    host_out = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    host_scores = torch.empty(T, dtype=torch.float32).pin_memory()
    host_tscores = torch.empty(pool.max_traces, dtype=torch.float32).pin_memory()
    host_npruned = torch.empty(1, dtype=torch.int32).pin_memory()
    stream = torch.cuda.current_stream()
    attn_events = []

    ids_host = list(ids)

    # the logical layers as runs of consecutive resident layers (one run unless fewer layers are resident than the model has)
    layer_runs = [(l0, min(phys_layers, L - l0)) for l0 in range(0, L, phys_layers)]

    q_stage = torch.empty((T, cfg.num_q_heads, cfg.head_dim), dtype=torch.bfloat16, device=dev)

    def hot_path(s, time_attn=False, out=out, step_scores=step_scores, layer_calls=None):
        """One decode step.  layer_calls: None = every run of resident layers through one decode_attention_layers call
        (all layers' queries at hand); "plain" = one decode_attention call per layer, as an engine makes them whose
        query of layer l + 1 is computed from the output of layer l; "dependent" = the same, each layer's query
        written by a stand-in kernel directly before the call and the attention launched as that kernel's
        programmatic dependent (decode_attention_dependent)."""
        pool.append_kv(ids_dev, 1, s["k"], s["v"])
        append_log.append((ids_host, 1))
        if layer_calls is None:
            for l0, nl in layer_runs:
                if time_attn:
                    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                # all layers of the run in one call: each launch a programmatic dependent of the one before it
                pool.decode_attention_layers(0, s["q"][l0:l0 + nl], v["block_table"], v["seq_lens"], out[l0:l0 + nl])
                if time_attn:
                    e1.record(stream); attn_events.append((e0, e1, nl))
        elif layer_calls == "plain":
            for l in range(L):
                pool.decode_attention(l % phys_layers, s["q"][l], v["block_table"], v["seq_lens"], out[l])
        elif layer_calls == "plain_after_producer":
            for l in range(L):
                torch.mul(s["q"][l], 1, out=q_stage)            # the same stand-in, the attention launched the ordinary way
                pool.decode_attention(l % phys_layers, q_stage, v["block_table"], v["seq_lens"], out[l])
        else:
            for l in range(L):
                torch.mul(s["q"][l], 1, out=q_stage)            # stands in for the projection kernel that produces q
                pool.decode_attention_dependent(l % phys_layers, q_stage, v["block_table"], v["seq_lens"], out[l])
        pool.score_steps(s["h"], s["m"], None, wts, step_scores)
        pool.prune_if_saturated(None, cfg.threshold, cfg.keep_frac)

    def timed_steps(n, **kw):
        """ms per step over n steps (two untimed ones first), CUDA events on the launching stream."""
        for i in range(2):
            hot_path(sets[i % NSETS], **kw)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(n):
            hot_path(sets[i % NSETS], **kw)
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    def make_e2e():
        """Returns run(n_steps): n_steps steps whose inputs start in pinned host memory and whose results end there,
        software-pipelined the way a serving loop would: while step i computes, the copy engines bring in the inputs of step i + 1 and take
        out the results of step i - 1 (two sets of device and host buffers); the host reads a step's results one step
        late.  Every step's copies happen inside the region that is timed; the buffers are set up here, outside it."""
        h2d_s, d2h_s = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        keys = ("q", "k", "v", "h", "m")
        dst = [{k: torch.empty_like(sets[0][k]) for k in keys} for _ in range(2)]
        outs = [out, torch.empty_like(out)]
        sc = [step_scores, torch.empty_like(step_scores)]
        ts = [torch.empty(pool.max_traces, dtype=torch.float32, device=dev) for _ in range(2)]
        npr = [torch.empty(1, dtype=torch.int32, device=dev) for _ in range(2)]
        host = [dict(out=host_out, sc=host_scores, ts=host_tscores, n=host_npruned),
                dict(out=torch.empty_like(host_out).pin_memory(), sc=torch.empty_like(host_scores).pin_memory(),
                     ts=torch.empty_like(host_tscores).pin_memory(), n=torch.empty_like(host_npruned).pin_memory())]
        in_done = [torch.cuda.Event() for _ in range(2)]
        comp_done = [torch.cuda.Event() for _ in range(2)]
        out_done = [torch.cuda.Event() for _ in range(2)]

        def run(n_steps):
            fetch(0)
            for i in range(n_steps):
                p = i % 2
                if i + 1 < n_steps:
                    fetch(i + 1)
                stream.wait_event(in_done[p])
                if i >= 2:
                    stream.wait_event(out_done[p])      # the results of step i - 2 have left these buffers
                hot_path(dst[p], out=outs[p], step_scores=sc[p])
                ts[p].copy_(v["trace_scores"], non_blocking=True)
                npr[p].copy_(pool.n_pruned, non_blocking=True)
                comp_done[p].record(stream)
                with torch.cuda.stream(d2h_s):
                    d2h_s.wait_event(comp_done[p])
                    host[p]["out"].copy_(outs[p], non_blocking=True)
                    host[p]["sc"].copy_(sc[p], non_blocking=True)
                    host[p]["ts"].copy_(ts[p], non_blocking=True)
                    host[p]["n"].copy_(npr[p], non_blocking=True)
                    out_done[p].record(d2h_s)
                if i >= 1:
                    out_done[1 - p].synchronize()       # the host has step i - 1's results
            out_done[(n_steps - 1) % 2].synchronize()
            torch.cuda.synchronize()

        def fetch(i):                                   # inputs of step i -> device set i % 2
            p = i % 2
            with torch.cuda.stream(h2d_s):
                if i >= 2:
                    h2d_s.wait_event(comp_done[p])      # step i - 2 has finished reading this set
                for k in keys:
                    dst[p][k].copy_(sets[i % NSETS]["host"][k], non_blocking=True)
                in_done[p].record(h2d_s)

        return run

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing
    for i in range(Wm):
        hot_path(sets[i % NSETS])
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for i in range(K):
        hot_path(sets[i % NSETS], time_attn=True)
    ev1.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = ev0.elapsed_time(ev1)
    attn_run_ms = [a.elapsed_time(b) for a, b, _ in attn_events]
    attn_ms = [t / nl for t, (_, _, nl) in zip(attn_run_ms, attn_events)]     # per launch, within its run of layers
    attn_launches = sum(nl for _, _, nl in attn_events)
    # the same kernel launched alone (plain decode_attention calls, one event pair each), for comparison; launches
    # on their own get the library's default balance
    pool.set_attention_balance(LIB_BALANCE)
    iso = []
    for i in range(2 + 12):                                              # two untimed launches first
        l = i % phys_layers
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        pool.decode_attention(l, sets[0]["q"][l], v["block_table"], v["seq_lens"], out[l])
        e1.record(stream)
        if i >= 2:
            iso.append((e0, e1))
    torch.cuda.synchronize()
    iso_ms = float(np.mean([a.elapsed_time(b) for a, b in iso]))
    pool.set_attention_balance(step_balance)
    # whole steps the way a layer-by-layer engine would make them (outside `value`; single-GPU runs only)
    per_layer_ms = dep_layer_ms = prod_layer_ms = None
    probe = None
    if world == 1 and not args.no_aux:
        pool.set_attention_balance(LIB_BALANCE)                          # one call per layer: launches on their own
        per_layer_ms = timed_steps(K, layer_calls="plain")
        prod_layer_ms = timed_steps(K, layer_calls="plain_after_producer")
        dep_layer_ms = timed_steps(K, layer_calls="dependent")
        pool.set_attention_balance(step_balance)
        probe = read_stream_ceiling(pool, cfg, dev, L)
    err_code, err_mask = pool.last_error()
    n_live = pool.stats()["live_traces"]
    seq_now = v["seq_lens"][:T].cpu().numpy().astype(np.int64)

    # ---- end to end: host buffers in, host results out, every step
    e2e = None
    if e2e_steps:
        e2e_run = make_e2e()
        e2e_run(Wm)
        barrier()
        t0 = time.perf_counter()
        e2e_run(e2e_steps)
        barrier()
        e2e_s = time.perf_counter() - t0
        h2d = sum(sets[0]["host"][k].numel() * sets[0]["host"][k].element_size() for k in ("q", "k", "v", "h", "m"))
        d2h = host_out.numel() * 4 + host_scores.numel() * 4 + host_tscores.numel() * 4 + 4
        e2e = (e2e_s, h2d, d2h)

    (ms_total, e2e_max), all_ok = R.max_over_ranks([ms_total, e2e[0] if e2e else 0.0], err_mask == 0 and n_live == T, dev)
    if e2e:
        e2e = (e2e_max, e2e[1], e2e[2])
    if world > 1:
        # every rank leaves the group at the same point; the CPU baseline and the measurements that follow the timed
        # steps belong to single-GPU runs (they would hold the other GPUs idle)
        dist.destroy_process_group()
        args.no_cpu_baseline = args.no_aux = True
    if rank != 0:
        return

    # ---- roofline of the dominant kernel (decode_attention of one layer)
    peak, peak_kind = measured_peaks()
    mid_suffix = seq_now - cfg.prefix_len - K // 2          # lengths at the middle of the timed region
    kv_bytes = H.unique_kv_bytes(cfg, cfg.prefix_len, mid_suffix)
    pages = int(np.sum(-(-(mid_suffix + cfg.prefix_len) // cfg.page_size)))
    algo_bytes = kv_bytes + T * cfg.num_q_heads * cfg.head_dim * (2 + 4) + pages * 4
    attn_avg_ms = float(np.sum(attn_run_ms)) / attn_launches
    achieved = algo_bytes / (attn_avg_ms * 1e-3) / 1e9
    traffic_ratio, traffic_src = attention_dram_traffic_ratio()
    value = R.whole_job_rate(T * K, world, ms_total * 1e-3)
    res = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic (seeded, drawn on device)",
        "config": {"workload": cfg.name, "traces": T, "layers": L, "layers_resident": phys_layers,
                   "q_heads": cfg.num_q_heads, "kv_heads": cfg.num_kv_heads, "head_dim": cfg.head_dim,
                   "page": cfg.page_size, "num_blocks": nb, "pool_gb": round(pool.kv_bytes / 1e9, 2),
                   "tokens_per_trace": int(np.mean(seq_now)), "threshold": cfg.threshold, "keep_frac": cfg.keep_frac,
                   "l2_policy": "inputs larger than L2 (%.1f GB of KV per layer call)" % (kv_bytes / 1e9),
                   "attention_balance": {"timed_steps_sixteenths": step_balance, "single_launches_sixteenths": LIB_BALANCE,
                                         "what": "share of every sequence's pages that warps fetch at run time "
                                                 "(kv_pool_set_attention_balance); the rest is dealt out in equal shares"},
                   "multi_gpu": "replicas only (one independent problem per GPU)", "fill_s": round(t_fill, 1)},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": "of " + peak_kind, "frac_of_nominal_8TBs": achieved / 8000.0,
                     "traffic": None if traffic_ratio is None else algo_bytes * traffic_ratio,
                     "traffic_source": traffic_src,
                     "kernel": "decode_attention_layers (attn_mma_kernel plus attn_merge_kernel, which combines the split partials), per layer",
                     "algorithmic_bytes_per_launch": algo_bytes, "avg_launch_ms": attn_avg_ms,
                     "min_launch_ms": float(np.min(attn_ms)), "launches_timed": attn_launches,
                     "how_timed": "CUDA events around each decode_attention_layers call (all layers of a step: every launch after "
                                  "the first is a programmatic dependent of the one before it, so launches overlap at layer "
                                  "boundaries); avg_launch_ms = elapsed / launches.  The peak is a copy (reads and writes) of one "
                                  "isolated launch; read_stream_ceiling gives the same device's read-only stream, isolated and chained.",
                     "isolated_launch": {"avg_launch_ms": iso_ms, "achieved": algo_bytes / (iso_ms * 1e-3) / 1e9,
                                         "frac": algo_bytes / (iso_ms * 1e-3) / 1e9 / peak,
                                         "what": "plain decode_attention calls timed one by one after the timed region"}},
        "kv_gbs": achieved,
        # what a caller gets that runs the model layer by layer (NextToken computes the query of layer l + 1 from the
        # output of layer l, so the 36 queries of a step are not at hand together): whole steps, one call per layer
        "per_layer_calls": None if per_layer_ms is None else {
            "what": "the same whole step with one decode_attention call per layer instead of one decode_attention_layers call",
            "ms_per_step": per_layer_ms, "value": T / (per_layer_ms * 1e-3), "unit": UNIT,
            "attention_gbs_upper": algo_bytes * L / (per_layer_ms * 1e-3) / 1e9,
            "frac": algo_bytes * L / (per_layer_ms * 1e-3) / 1e9 / peak,
            "dependent_on_q_producer": {
                "what": "each layer's q written by a stand-in kernel directly before the call; decode_attention_dependent "
                        "(scheduled behind that kernel, waits for it only in front of its first read of q)",
                "ms_per_step": dep_layer_ms, "value": T / (dep_layer_ms * 1e-3),
                "frac": algo_bytes * L / (dep_layer_ms * 1e-3) / 1e9 / peak,
                "ordinary_launch_after_the_same_stand_in_ms_per_step": prod_layer_ms},
            "note": "frac counts the whole step's time (append, scorer and trigger included) against the attention bytes"},
        "read_stream_ceiling": probe,
        # the same launches counted the way a per-trace kernel would see them (the shared prompt once per trace)
        "kv_gbs_logical": float(np.sum(seq_now - K // 2)) * cfg.bytes_per_token_layer / (attn_avg_ms * 1e-3) / 1e9,
        "attention_share_of_step": float(np.sum(attn_run_ms)) / ms_total,
        "gpu_launches": K * (1 + 2 * L + 1 + 1), "clocks": clocks,
        "status": {"device_error_mask": err_mask, "live_traces": n_live, "ok": all_ok},
    }
    if e2e:
        res["e2e"] = {"value": R.whole_job_rate(T * e2e_steps, world, e2e[0]), "unit": UNIT, "h2d_bytes_per_step": e2e[1],
                      "d2h_bytes_per_step": e2e[2], "ms_per_step": e2e[0] * 1e3 / e2e_steps}
    if not args.no_cpu_baseline:
        res["cpu_baseline"], res["sampled_parity"] = cpu_baseline_and_parity(pool, cfg, sets[(K - 1) % NSETS], out, L, phys_layers)
    if not args.no_aux:
        res["algorithm1_loop"] = algorithm1_measurement(pool, cfg, T, phys_layers, dev, wts, sets, append_log, ids_host,
                                                        ms_total / K if phys_layers == L else None)
        res["scorer"] = scorer_measurements(cfg, dev, rows=args.scorer_rows)
        res["append_kv"] = append_measurements(cfg, dev, min(phys_layers, 36))
        if args.workload == "c3":
            # last: this consumes the benchmark state (the pool ends with two live traces)
            cyc = prune_cycles(pool, cfg, nb, T, dev, wts, append_log, phys_layers, peak)
            res["prune_cycles"] = cyc["report"]
            if not args.no_cpu_baseline:
                res["prune_cycles"]["oracle_replay"] = replay_cycles_on_oracle(cfg, nb, T, max_pages, append_log, cyc["snapshots"])
    print(json.dumps(res))


def read_stream_ceiling(pool, cfg, dev, n_launches, reps=3):
    """step_read_stream_probe over one layer's worth of the pool's KV storage: the attention kernel's copy structure with
    no arithmetic, `n_launches` launches in a row, launched the ordinary way and chained as programmatic dependents."""
    import torch
    from paper_2601_09093_b200 import binding as B
    layer_bytes = pool.num_blocks * cfg.bytes_per_token_layer * cfg.page_size
    buf = pool.kv_storage[:layer_bytes]
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    peak, kind = measured_peaks()
    out = {"what": "cp.async.bulk rings of the attention kernel reading %.2f GB and dropping it, %d launches in a row" % (layer_bytes / 1e9, n_launches),
           "bytes_per_launch": layer_bytes}
    for name, chained in (("isolated", 0), ("chained", 1)):
        B.read_stream_probe(buf, n_launches, chained, err)
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); B.read_stream_probe(buf, n_launches, chained, err); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) / n_launches)
        ms = float(np.median(ts))
        out[name] = {"ms_per_launch": ms, "gbs": layer_bytes / (ms * 1e-3) / 1e9, "frac_of_copy_peak": layer_bytes / (ms * 1e-3) / 1e9 / peak}
    out["error_flag"] = int(err.item())
    return out


def blas_threads():
    """Threads numpy's BLAS uses for the oracle's products, as threadpoolctl reports them (None if unknown)."""
    try:
        from threadpoolctl import threadpool_info
        n = [int(p.get("num_threads", 0)) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else None
    except Exception:
        return None


def cpu_baseline_and_parity(pool, cfg, s, out, L, phys_layers, cpu_budget_s=12.0):
    """Times the oracle on a bounded sample of the benchmark's own state and checks the GPU against it.

    Sample: whole (trace, layer) attentions - all KV heads and query heads of a trace in one layer -
    taken round-robin over layers {last, first, middle, ...} and over all traces until about
    `cpu_budget_s` seconds of oracle time are spent.  The stored K/V rows are read back through
    kv_pool_read_kv so that the oracle sees the very bytes the kernel read.  CPU throughput is
    extrapolated to whole trace-decode-steps by the layer count.
    """
    import torch
    from oracle import attention as OA
    v = pool.views()
    T = cfg.n_traces
    layers = [L - 1, 0, L // 2] + [l for l in range(1, L - 1) if l != L // 2]
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    t_cpu, max_err, sum_err, cnt, done = 0.0, 0.0, 0.0, 0, 0
    wall0 = time.perf_counter()
    # the outputs of every layer for the inputs in `s`, recomputed the way the timed steps launch them (runs of
    # consecutive resident layers through decode_attention_layers) so that they are known to match these inputs
    for l0 in range(0, L, phys_layers):
        nl = min(phys_layers, L - l0)
        pool.decode_attention_layers(0, s["q"][l0:l0 + nl], v["block_table"], v["seq_lens"], out[l0:l0 + nl])
    torch.cuda.synchronize()
    for layer in layers[:L]:
        got_all = out[layer].cpu().numpy().astype(np.float64)
        q_all = s["q"][layer].float().cpu().numpy().astype(np.float64)
        for t in range(T):
            S = int(v["seq_lens"][t].item())
            K_ = np.empty((S, cfg.num_kv_heads, cfg.head_dim), dtype=np.float64)
            V_ = np.empty_like(K_)
            for h in range(cfg.num_kv_heads):
                k, vv = pool.read_kv(layer % phys_layers, h, v["block_table"][t], S)
                K_[:, h] = k.float().cpu().numpy(); V_[:, h] = vv.float().cpu().numpy()
            t0 = time.perf_counter()
            want = OA.dense_decode_attention(q_all[t], K_, V_)
            t_cpu += time.perf_counter() - t0
            err = np.abs(got_all[t] - want)
            max_err = max(max_err, float(err.max())); sum_err += float(err.sum()); cnt += err.size
            done += 1
            if t_cpu >= cpu_budget_s or time.perf_counter() - wall0 > 90.0:
                break
        if t_cpu >= cpu_budget_s or time.perf_counter() - wall0 > 90.0:
            break
    value = done / (t_cpu * L)
    # the same oracle held to one thread, on a few of the same attentions (the last trace's K, V and q are still at hand)
    single = None
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            t0 = time.perf_counter()
            n1 = 0
            while time.perf_counter() - t0 < 2.0:
                OA.dense_decode_attention(q_all[t], K_, V_)
                n1 += 1
            single = n1 / ((time.perf_counter() - t0) * L)
    except Exception:
        pass
    threads = blas_threads()
    base = {"value": value, "unit": UNIT, "cores": threads or cores, "host_cores": cores, "blas_threads": threads,
            "single_thread_value": single, "kind": "oracle",
            "sample": "%d (trace, layer) attentions at full length, all heads (%.1f s of CPU), extrapolated to %d layers per step; "
                      "cores = the threads numpy's BLAS used; single_thread_value = the same oracle limited to one thread (2 s sample)"
                      % (done, t_cpu, L)}
    par = {"what": "decode_attention_layers (the timed launch configuration) vs fp64 oracle on read-back KV: %d (trace, layer) pairs, all heads" % done,
           "max_abs_err": max_err, "mean_abs_err": sum_err / cnt, "tolerance": {"max": 1e-2, "mean": 1e-3},
           "ok": bool(max_err <= 1e-2 and sum_err / cnt <= 1e-3)}
    return base, par



# ---------------------------------------------------------------------------------------------
ALG1_ITERATIONS = 6                 # iterations of the directly launched run on the 36-layer workloads
ALG1_ITERATIONS_ONE_LAYER = 40      # ... and on the one-layer workloads, where the end-of-call round trip would weigh on six
ALG1_GRAPH_ITERATIONS = 40          # iterations of the recorded-iteration run on the one-layer workloads (6 on the others)


def algorithm1_measurement(pool, cfg, T, phys_layers, dev, wts, sets, append_log, ids_host, ms_per_step_python):
    """The same decode step driven by the library's own loop (algorithm1_run: one C call for all iterations, step-end
    flags taken from sampled token ids, completion handling included) instead of one Python call per kernel group.
    No trace samples the end-of-sequence token and the trigger stays quiet, so the work per iteration equals a step
    of the timed region.  Also times detect_step_ends alone on 4M tokens."""
    import torch
    from paper_2601_09093_b200 import binding as B, workloads as W
    vocab = W.synthetic_vocab(cfg.seed, 32000, step_end_frac=0.01)
    table = B.step_end_table_from_vocab(vocab)
    ends = np.flatnonzero(table.numpy())
    n_direct = ALG1_ITERATIONS_ONE_LAYER if phys_layers == 1 else ALG1_ITERATIONS
    toks = np.stack([W.token_ids(cfg.seed, T, len(vocab), ends, cfg.boundary_density, sub=500 + i)
                     for i in range(n_direct + 2 + ALG1_GRAPH_ITERATIONS + 2)])
    toks[toks == 0] = 1                                            # id 0 is the end-of-sequence token here: nobody completes
    table_d, toks_d = table.to(dev), torch.from_numpy(toks).to(dev)
    q = torch.stack([s["q"][:phys_layers] for s in sets]).contiguous()
    k = torch.stack([s["k"] for s in sets]).contiguous()
    v = torch.stack([s["v"] for s in sets]).contiguous()
    h = torch.stack([s["h"] for s in sets]).contiguous()
    answers = torch.zeros(T, dtype=torch.int32, device=dev)
    attn_out = torch.empty((phys_layers, T, cfg.num_q_heads, cfg.head_dim), dtype=torch.float32, device=dev)

    def run(tok, n, graphs=False):
        r = pool.algorithm1_run(tok, 0, table_d, answers, q, k, v, h, wts, cfg.threshold, cfg.keep_frac,
                                check_every=n, attn_out=attn_out, use_graphs=graphs)
        for _ in range(n):
            append_log.append((ids_host, 1))
        return r

    run(toks_d[:2], 2)                                              # warm-up
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    r = run(toks_d[2:2 + n_direct], n_direct)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n_direct
    # the same loop with each ring slot's iteration recorded as a CUDA graph (on a stream that can be captured); the
    # timed call records its two graphs itself, so that cost is inside the figure
    n_g = ALG1_GRAPH_ITERATIONS if phys_layers == 1 else 6
    base = 2 + n_direct
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run(toks_d[base:base + 2], 2, graphs=True)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(side)
        rg = run(toks_d[base + 2:base + 2 + n_g], n_g, graphs=True)
        g1.record(side)
    torch.cuda.synchronize()
    torch.cuda.current_stream().wait_stream(side)
    ms_g = g0.elapsed_time(g1) / n_g
    # the loop's attention launches follow one another as programmatic dependents; the outputs of its last iteration
    # must be, bit for bit, what one plain decode_attention call per layer gives on the same (unchanged) state
    vv = pool.views()
    q_last = q[(n_g - 1) % len(sets)]
    same = True
    for l in range(phys_layers):
        direct = pool.decode_attention(l, q_last[l], vv["block_table"], vv["seq_lens"])
        same = same and bool(torch.equal(direct, attn_out[l]))
    # step-end detection alone
    n_tok = 1 << 22
    big = torch.from_numpy(W.token_ids(cfg.seed, n_tok, len(vocab), ends, cfg.boundary_density, sub=77)).to(dev)
    mask = torch.empty(n_tok, dtype=torch.uint8, device=dev)
    for _ in range(3):
        pool.detect_step_ends(big, table_d, mask)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(11)]
    ev[0].record()
    for i in range(10):
        pool.detect_step_ends(big, table_d, mask)
        ev[i + 1].record()
    torch.cuda.synchronize()
    det_ms = float(np.median([ev[i].elapsed_time(ev[i + 1]) for i in range(10)]))
    code, bits = pool.last_error()
    return {"iterations": r["iterations"], "ms_per_iteration": ms, "trace_decode_steps_per_s": T / (ms * 1e-3),
            "vs_python_driven_step": None if ms_per_step_python is None else ms_per_step_python / ms,
            "layers_per_iteration": phys_layers, "launches_per_iteration": 3 + 2 * phys_layers,
            "live_left": r["live_left"], "n_evicted": r["n_evicted"], "n_finished": r["n_finished"],
            "recorded_iterations": {"iterations": rg["iterations"], "ms_per_iteration": ms_g,
                                    "trace_decode_steps_per_s": T / (ms_g * 1e-3), "vs_direct_launches": ms / ms_g,
                                    "live_left": rg["live_left"]},
            "attention_outputs_equal_plain_calls": same,
            "detect_step_ends": {"tokens": n_tok, "us_per_call": det_ms * 1e3, "tokens_per_s": n_tok / (det_ms * 1e-3),
                                 "gbs": n_tok * 5 / (det_ms * 1e-3) / 1e9},
            "device_error_mask": bits}


def scorer_measurements(cfg, dev, rows=65536, reps=20, all_rows_density=1.0):
    """score_steps timed alone (CUDA events around each call, median of `reps`) on three shapes of one scorer:
    a decode step (one row per trace, Bernoulli step-end flags), the batched shape (1024 rows per trace at the
    same density) and `rows` rows that all end a step (scoring every step of many finished traces at once)."""
    import torch
    from paper_2601_09093_b200 import binding as B, harness as H, workloads as W
    T = cfg.n_traces
    (W1b, _), (b1b, _), (w2b, _), b2 = W.scorer_weights(cfg, bias_std=0.05)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16", dev), H.to_device(b1b, "bf16", dev), H.to_device(w2b, "bf16", dev), b2, B.STEP_BF16)
    gen = torch.Generator(device=dev); gen.manual_seed(cfg.seed + 55)
    shapes = [("decode", T, cfg.boundary_density), ("batched", T * 1024, cfg.boundary_density), ("all_rows", rows, all_rows_density)]
    Mmax = max(m for _, m, _ in shapes)
    pool = H.make_pool(W.scaled(cfg, num_layers=1), 8, 4, T, max_score_rows=Mmax, device=dev)
    hid = torch.randn((Mmax, cfg.scorer_D), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    rt = (torch.arange(Mmax, device=dev) % T).to(torch.int32)
    out = torch.empty(Mmax, dtype=torch.float32, device=dev)
    peak, kind = measured_peaks("bf16_tflops", 1590.0)
    res = {"D": cfg.scorer_D, "m": cfg.scorer_m, "unit": "boundary rows scored per second (scorer calls/s)",
           "flops_per_row": 2 * cfg.scorer_m * (cfg.scorer_D + 1), "bf16_peak_tflops": peak, "peak_kind": "of " + kind}
    for name, M, density in shapes:
        if density >= 1.0:
            mask = torch.ones(M, dtype=torch.uint8, device=dev)
        else:
            mask = torch.from_numpy(W.boundary_mask(cfg, M, sub=900, density=density)).to(dev)
            if int(mask.sum().item()) == 0:
                mask[0] = 1
        for _ in range(3):
            pool.score_steps(hid[:M], mask, rt[:M], wts, out[:M])
        info = pool.score_launch_info()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        ev[0].record()
        for i in range(reps):
            pool.score_steps(hid[:M], mask, rt[:M], wts, out[:M])
            ev[i + 1].record()
        torch.cuda.synchronize()
        ms = float(np.median([ev[i].elapsed_time(ev[i + 1]) for i in range(reps)]))
        nbr = info["n_rows"]
        tfl = nbr * res["flops_per_row"] / (ms * 1e-3) / 1e12
        res[name] = {"rows": M, "boundary_rows": nbr, "us_per_call": ms * 1e3, "rows_per_s": nbr / (ms * 1e-3),
                     "tflops": tfl, "frac_of_bf16_peak": tfl / peak,
                     "first_layer": ("tcgen05, %d units per CTA" % info["tc_units"]) if info["tc_units"] else "cuda cores"}
        if name == "decode":
            # a call this short is bound by the host's launch rate when timed back to back: queue the calls behind a
            # kernel that keeps the GPU busy, so that the events see the device's own time; and once more with the L2
            # flushed before every call (in a decode step the attention launches have just streamed gigabytes through it)
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
            for cold in (False, True):
                ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
                torch.cuda._sleep(int(2e7))
                for a_, b_ in ev:
                    if cold:
                        flush.zero_()
                    a_.record(); pool.score_steps(hid[:M], mask, rt[:M], wts, out[:M]); b_.record()
                torch.cuda.synchronize()
                res[name]["us_per_call_device" + ("_cold_l2" if cold else "")] = float(np.median([a_.elapsed_time(b_) for a_, b_ in ev])) * 1e3
            del flush
    code, mask_bits = pool.last_error()
    res["device_error_mask"] = mask_bits
    pool.close()
    # one optimisation step of the scorer at the paper's batch size (128 labelled step-end hidden states)
    Bt = 128
    tr = B.ScorerTrainer(wts.W1.float(), wts.b1.float(), wts.w2.float(), wts.b2, batch=Bt, pos_weight=2.0)
    labels = (torch.arange(Bt, device=dev) % 3 == 0).float()
    for _ in range(3):
        tr.step(hid[:Bt], labels)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    ev[0].record()
    for i in range(reps):
        tr.step(hid[:Bt], labels)
        ev[i + 1].record()
    torch.cuda.synchronize()
    ms = float(np.median([ev[i].elapsed_time(ev[i + 1]) for i in range(reps)]))
    n_par = cfg.scorer_m * cfg.scorer_D + 2 * cfg.scorer_m + 1
    res["train_step"] = {"batch": Bt, "us_per_step": ms * 1e3, "loss": float(tr.loss.item()),
                         "gflops": 2 * 2.0 * Bt * cfg.scorer_m * cfg.scorer_D / (ms * 1e-3) / 1e9,
                         "adam_bytes": n_par * 28, "launches": 5}
    return res


WINDOW = 16                         # whole decode steps timed before each saturation point and after each prune


def append_measurements(cfg, dev, layers, reps=20):
    """append_kv alone on a pool of its own: the decode step's call (one new token for every trace, all `layers`
    layers), timed on the device with the calls queued behind a kernel that keeps the GPU busy, and a bulk call
    (32 tokens per trace), whose bytes (read + written) are set against the measured copy peak."""
    import torch
    from paper_2601_09093_b200 import harness as H, workloads as W
    T = cfg.n_traces
    c = W.scaled(cfg, num_layers=layers)
    bulk = 32
    pages = T * (2 + (reps + 8) * bulk // c.page_size + (2 * reps + 40) // c.page_size + 2) + 8
    pool = H.make_pool(c, pages, pages // T + 2, T, device=dev)
    gen = torch.Generator(device=dev); gen.manual_seed(cfg.seed + 99)
    rnd = lambda *shape: torch.randn(shape, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    ids = torch.tensor(pool.fork_prefix(T, 16, rnd(layers, c.num_kv_heads, 16, c.head_dim), rnd(layers, c.num_kv_heads, 16, c.head_dim)),
                       dtype=torch.int32, device=dev)
    k1, v1 = rnd(T, 1, layers, c.num_kv_heads, c.head_dim), rnd(T, 1, layers, c.num_kv_heads, c.head_dim)
    kb, vb = rnd(T, bulk, layers, c.num_kv_heads, c.head_dim), rnd(T, bulk, layers, c.num_kv_heads, c.head_dim)
    peak, kind = measured_peaks()
    res = {"traces": T, "layers": layers}
    for name, kk, vv, n_tok in (("one_token", k1, v1, 1), ("bulk_32_tokens", kb, vb, bulk)):
        for _ in range(3):
            pool.append_kv(ids, n_tok, kk, vv)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        torch.cuda._sleep(int(2e7))
        for a_, b_ in ev:
            a_.record(); pool.append_kv(ids, n_tok, kk, vv); b_.record()
        torch.cuda.synchronize()
        us = float(np.median([a_.elapsed_time(b_) for a_, b_ in ev])) * 1e3
        moved = 2 * 2 * kk.numel() * 2                       # K and V, read and written, two bytes each
        res[name] = {"us_per_call_device": us, "bytes_read_and_written": moved, "gbs": moved / us / 1e3,
                     "frac_of_copy_peak": moved / us / 1e3 / peak}
    res["device_error_mask"] = pool.last_error()[1]
    pool.close()
    return res


def prune_cycles(pool, cfg, nb, T, dev, wts, append_log, phys_layers, hbm_peak, n_cycles=5):
    """The memory-saturated workload proper, continued from the benchmark state: the live traces grow until the
    pool reaches the trigger (used + need > floor(threshold * total)), every live trace gets a fresh step score,
    prune_if_saturated keeps the top half and reclaims the rest; five times, 64 -> 2 live traces.  Growth is by bulk
    append_kv up to WINDOW + 1 tokens short of each saturation point; the last WINDOW steps before it and the first
    WINDOW steps after each prune are whole decode steps through the normal step path (append_kv of one token,
    decode_attention_layers over all layers, score_steps, prune_if_saturated), timed with CUDA events.  At the
    saturation point itself single decode_attention launches and the prune call are timed.  Returns the report and,
    for the oracle's replay, what the GPU decided and left behind at each cycle."""
    import torch
    v = pool.views()
    P, L = cfg.page_size, phys_layers
    limit = math.floor(float(np.float32(cfg.threshold)) * nb)
    per_tok = L * cfg.num_kv_heads * cfg.head_dim                       # K (or V) elements of one token
    gen = torch.Generator(device=dev); gen.manual_seed(cfg.seed + 77)
    buf_elems = 1 << 27                                                  # 256 MB of K and of V per append call
    kbuf = torch.randn(buf_elems, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    vbuf = torch.randn(buf_elems, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    hid = torch.randn((T, cfg.scorer_D), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    q = torch.randn((T, cfg.num_q_heads, cfg.head_dim), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    q_step = torch.randn((L, T, cfg.num_q_heads, cfg.head_dim), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty((T, cfg.num_q_heads, cfg.head_dim), dtype=torch.float32, device=dev)
    out_step = torch.empty((L, T, cfg.num_q_heads, cfg.head_dim), dtype=torch.float32, device=dev)
    step_scores = torch.empty(T, dtype=torch.float32, device=dev)
    step_mask = torch.from_numpy(W_boundary(cfg, T)).to(dev)
    stream = torch.cuda.current_stream()

    def window(live, live_h, n_steps):
        """n_steps whole decode steps of the live traces; returns ms per step."""
        shape = (len(live_h), 1, L, cfg.num_kv_heads, cfg.head_dim)
        mask = step_mask & v["live"][:T]
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_steps):
            pool.append_kv(live, 1, kbuf[: len(live_h) * per_tok].view(shape), vbuf[: len(live_h) * per_tok].view(shape))
            append_log.append((live_h, 1))
            pool.decode_attention_layers(0, q_step, v["block_table"], v["seq_lens"], out_step)
            pool.score_steps(hid, mask, None, wts, step_scores)
            pool.prune_if_saturated(None, cfg.threshold, cfg.keep_frac)
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n_steps

    report, snaps = [], []
    for cyc in range(n_cycles):
        live_h = torch.nonzero(v["live"][:T]).flatten().cpu().tolist()
        n_live = len(live_h)
        if n_live < 4:                                                   # the block table is sized for four survivors
            break
        live = torch.tensor(live_h, dtype=torch.int32, device=dev)
        used = pool.stats()["used"]
        S = int(v["seq_lens"][live_h[0]].item())                         # survivors have equal lengths
        new_pages = (limit - used) // n_live
        n_tok = (-(-S // P) + new_pages) * P - S                         # tokens to the saturation point
        n_win = WINDOW if n_tok > WINDOW + 1 else 0
        c_max = max(1, buf_elems // (n_live * per_tok))
        left = n_tok - n_win - (1 if n_win else 0)
        while left > 0:
            c = min(left, c_max)
            shape = (n_live, c, L, cfg.num_kv_heads, cfg.head_dim)
            pool.append_kv(live, c, kbuf[: n_live * c * per_tok].view(shape), vbuf[: n_live * c * per_tok].view(shape))
            append_log.append((live_h, c))
            left -= c
        ms_before = None
        if n_win:
            # the last WINDOW steps before saturation (the trigger is evaluated in each and stays quiet), then the
            # token that brings the pool to the trigger
            ms_before = window(live, live_h, n_win)
            shape = (n_live, 1, L, cfg.num_kv_heads, cfg.head_dim)
            pool.append_kv(live, 1, kbuf[: n_live * per_tok].view(shape), vbuf[: n_live * per_tok].view(shape))
            append_log.append((live_h, 1))
        quiet = int(pool.n_pruned.item()) == 0 if n_win else True
        # decode attention at the saturation point (dead traces have length 0)
        n_att = 6
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_att + 1)]
        for l in range(2):
            pool.decode_attention(l % L, q, v["block_table"], v["seq_lens"], out)
        ev[0].record()
        for l in range(n_att):
            pool.decode_attention((2 + l) % L, q, v["block_table"], v["seq_lens"], out)
            ev[l + 1].record()
        torch.cuda.synchronize()
        att_ms = float(np.mean([ev[i].elapsed_time(ev[i + 1]) for i in range(n_att)]))
        tokens = S + n_tok
        kv_bytes = (cfg.prefix_len + n_live * (tokens - cfg.prefix_len)) * cfg.bytes_per_token_layer
        # a fresh score for every live trace, then the prune
        mask = v["live"][:T].clone()
        pool.score_steps(hid, mask, None, wts, step_scores)
        scores_h = v["trace_scores"].cpu().numpy().copy()
        st0 = pool.stats()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        # keep the GPU busy while the prune launch is enqueued, so that the events bracket the kernel and not the
        # host's launch latency (the stats() above drained the stream)
        pool.decode_attention(0, q, v["block_table"], v["seq_lens"], out)
        e0.record()
        pid, npr = pool.prune_if_saturated(None, cfg.threshold, cfg.keep_frac)
        e1.record()
        torch.cuda.synchronize()
        n_pruned = int(npr.item())
        st1 = pool.stats()
        fc = int(v["free_count"].item())
        snaps.append(dict(scores=scores_h, pruned=pid[:n_pruned].cpu().tolist(), free_list=v["free_list"][:fc].cpu().numpy(),
                          refcount=v["refcount"].cpu().numpy(), seq_lens=v["seq_lens"].cpu().numpy(),
                          live=v["live"].cpu().numpy(), block_table=v["block_table"].cpu().numpy(), log_pos=len(append_log)))
        # no waiting queue: every survivor's next token must find a block - the first WINDOW steps after the prune
        surv_h = torch.nonzero(v["live"][:T]).flatten().cpu().tolist()
        surv = torch.tensor(surv_h, dtype=torch.int32, device=dev)
        ms_after = window(surv, surv_h, WINDOW)
        code, bits = pool.last_error()
        report.append({"cycle": cyc + 1, "live_before": n_live, "live_after": st1["live_traces"], "tokens_per_trace": tokens,
                       "used_blocks_before": st0["used"], "blocks_reclaimed": st0["used"] - st1["used"],
                       "prune_us": e0.elapsed_time(e1) * 1e3, "blocks_reclaimed_per_s": (st0["used"] - st1["used"]) / (e0.elapsed_time(e1) * 1e-3),
                       "attention_ms_per_layer": att_ms, "attention_kv_gbs": kv_bytes / (att_ms * 1e-3) / 1e9,
                       "attention_frac_of_hbm_peak": kv_bytes / (att_ms * 1e-3) / 1e9 / hbm_peak,
                       "steps_before_saturation": None if ms_before is None else {
                           "steps": n_win, "ms_per_step": ms_before, "trace_decode_steps_per_s": n_live / (ms_before * 1e-3),
                           "kv_gbs": kv_bytes * L / (ms_before * 1e-3) / 1e9, "trigger_stayed_quiet": quiet},
                       "steps_after_prune": {
                           "steps": WINDOW, "ms_per_step": ms_after, "trace_decode_steps_per_s": len(surv_h) / (ms_after * 1e-3),
                           "kv_gbs": (cfg.prefix_len + len(surv_h) * (tokens + WINDOW // 2 - cfg.prefix_len)) * cfg.bytes_per_token_layer * L / (ms_after * 1e-3) / 1e9},
                       "survivors_scheduled_next_token": bits == 0, "device_error_mask": bits})
    return {"report": {"threshold": cfg.threshold, "keep_frac": cfg.keep_frac, "window_steps": WINDOW,
                       "what": "per cycle: WINDOW whole decode steps (all layers) timed just before the saturation point and just "
                               "after the prune; single attention launches and the prune call timed at the saturation point",
                       "cycles": report}, "snapshots": snaps}


def W_boundary(cfg, T):
    from paper_2601_09093_b200 import workloads as W
    return W.boundary_mask(cfg, T, sub=4242)


def replay_cycles_on_oracle(cfg, nb, T, max_pages, append_log, snaps):
    """The oracle's pool (bookkeeping only) is taken through the run's every append_kv call and, at each cycle, is
    given the GPU's trace scores; its evicted set, free list, reference counts, lengths, live flags and block table
    must equal what the GPU left, bit for bit.  Part of the CPU leg: the oracle's prune is timed too."""
    from oracle.kv_pool import KVPoolOracle
    o = KVPoolOracle(cfg.num_layers, cfg.num_kv_heads, cfg.head_dim, cfg.page_size, nb, T, max_pages, store_payload=False)
    o.fork_prefix(T, cfg.prefix_len)
    pos, ok, cpu_us, first_bad = 0, True, [], None
    for k, sn in enumerate(snaps):
        for ids, n in append_log[pos:sn["log_pos"]]:
            o.append_kv(ids, n)
        pos = sn["log_pos"]
        t0 = time.perf_counter()
        got = o.prune_if_saturated(sn["scores"], cfg.threshold, cfg.keep_frac)
        cpu_us.append((time.perf_counter() - t0) * 1e6)
        same = (got == sn["pruned"] and o.free_list == sn["free_list"].tolist()
                and np.array_equal(o.refcount, sn["refcount"]) and np.array_equal(o.seq_lens, sn["seq_lens"])
                and np.array_equal(o.live, sn["live"].astype(bool)) and np.array_equal(o.block_table, sn["block_table"]))
        if not same and first_bad is None:
            first_bad = k + 1
        ok = ok and same
    return {"what": "evicted ids, free list, refcounts, lengths, live flags and block table after each prune, bit-exact "
                    "against the oracle replaying all %d append_kv calls with the GPU's scores" % len(append_log),
            "ok": bool(ok), "first_mismatching_cycle": first_bad, "oracle_prune_us": cpu_us, "status_bits": int(o.status)}


# ---------------------------------------------------------------------------------------------
def scorer_shape(name):
    """The configuration whose scorer (D, m) the scorer workload uses; the paper's 4B and 14B-class models have
    hidden sizes 2560 and 5120 with the same 512-unit scorer."""
    from paper_2601_09093_b200 import workloads as W
    if name == "d2560":
        return W.scaled(W.C1, name="scorer-D2560-m512", scorer_D=2560)
    if name == "d5120":
        return W.scaled(W.C1, name="scorer-D5120-m512", scorer_D=5120)
    return {"c1": W.C1, "c4": W.C4}[name]


def run_scorer(args):
    """`--workload scorer`: score_steps alone on a large batch of step-end hidden states (every step of many
    finished traces scored at once).  The line's roofline is the tensor-core one of the first-layer GEMM."""
    import torch
    from paper_2601_09093_b200 import binding as B, ranks as R, workloads as W
    from paper_2601_09093_b200 import build as _build
    rank, local_rank, world = R.rank_env()
    if rank == 0:
        _build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    B.lib()
    cfg = scorer_shape(args.scorer_shape)
    K = max(args.steps, 3)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    m = scorer_measurements(cfg, dev, rows=args.scorer_rows, reps=K, all_rows_density=args.scorer_density)
    clocks = sampler.stop() if rank == 0 else None
    a = m["all_rows"]
    (a["us_per_call"],), _ = R.max_over_ranks([a["us_per_call"]], m["device_error_mask"] == 0, dev)
    a["rows_per_s"] = a["boundary_rows"] / (a["us_per_call"] * 1e-6)
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return
    flops = a["boundary_rows"] * m["flops_per_row"]
    res = {"metric": "scorer calls/s (step-end hidden states scored per second)", "value": R.whole_job_rate(a["boundary_rows"], world, a["us_per_call"] * 1e-6),
           "unit": "rows/s", "n_gpus": world, "steps": K, "warmup": 3, "ms_per_step": a["us_per_call"] * 1e-3,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
           "data": "synthetic (seeded, drawn on device)",
           "config": {"workload": "scorer-batched-%s" % cfg.name, "rows": a["rows"], "boundary_rows": a["boundary_rows"],
                      "D": cfg.scorer_D, "m": cfg.scorer_m, "first_layer": a["first_layer"],
                      "l2_policy": "inputs larger than L2 (%.0f MB of hidden states per call)" % (a["rows"] * cfg.scorer_D * 2 / 1e6)},
           "roofline": {"bound": "tensor", "achieved": a["tflops"], "peak": m["bf16_peak_tflops"], "unit": "TFLOP/s",
                        "frac": a["frac_of_bf16_peak"], "peak_kind": m["peak_kind"] + " (burst: the call is timed alone)",
                        "traffic": None, "kernel": "score_steps (compact + score_tc_kernel + finish), whole call",
                        "algorithmic_flops_per_launch": flops},
           "scorer": m, "gpu_launches": 3 * K, "clocks": clocks}
    print(json.dumps(res))


# ---------------------------------------------------------------------------------------------
def run_append(args):
    """`--workload append`: append_kv alone - the 64-trace, 36-layer layout; `--steps` calls of each kind are timed
    (the pool grows with that number: 2 steps hold 4 GB, the default 20 hold 10 GB)."""
    import torch
    from paper_2601_09093_b200 import ranks as R, workloads as W
    from paper_2601_09093_b200 import build as _build
    rank, local_rank, world = R.rank_env()
    if rank != 0:
        return
    _build.build()
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    m = append_measurements(W.C3, dev, W.C3.num_layers, reps=max(args.steps, 2))
    b = m["bulk_32_tokens"]
    print(json.dumps({"metric": "append_kv_bulk_bytes_per_s", "value": b["gbs"], "unit": "GB/s", "n_gpus": 1, "steps": max(args.steps, 2),
                      "warmup": 3, "ms_per_step": b["us_per_call_device"] * 1e-3, "higher_is_better": True, "scaling": "weak",
                      "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded, drawn on device)",
                      "config": {"workload": "append_kv on the 64-trace 36-layer layout", "l2_policy": "bulk call: 604 MB moved per call"},
                      "append_kv": m, "gpu_launches": 2 * (max(args.steps, 2) + 3)}))


# ---------------------------------------------------------------------------------------------
def run_prefix(args):
    """`--workload prefix`: decode_attention and decode_attention_shared_prefix on the same state - 64 traces of the
    8B layout whose shared prompt is long against what each trace generated (the regime the paper's workloads are
    NOT in: there the prompt is a few hundred tokens of tens of thousands).  One layer; single GPU."""
    import torch
    from paper_2601_09093_b200 import binding as B, harness as H, ranks as R, workloads as W
    from paper_2601_09093_b200 import build as _build
    rank, local_rank, world = R.rank_env()
    if rank != 0:
        return
    _build.build()
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    B.lib()
    cfg = W.scaled(W.C1, name="prefix-heavy-1layer", prefix_len=args.prefix_len, suffix_lo=1, suffix_hi=args.suffix_max)
    T, P = cfg.n_traces, cfg.page_size
    suffix = W.suffix_lengths(cfg)
    pp = cfg.prefix_len // P
    pages = pp + int(sum(-(-(cfg.prefix_len % P + int(x)) // P) for x in suffix))
    pool = H.make_pool(cfg, pages + 64, -(-(cfg.prefix_len + int(suffix.max())) // P) + 2, T, device=dev)
    H.fill_random_device(pool, cfg, suffix, seed=cfg.seed)
    v = pool.views()
    gen = torch.Generator(device=dev); gen.manual_seed(cfg.seed + 1)
    q = torch.randn((T, cfg.num_q_heads, cfg.head_dim), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    out_a = torch.empty((T, cfg.num_q_heads, cfg.head_dim), dtype=torch.float32, device=dev)
    out_b = torch.empty_like(out_a)
    prefix_blocks = v["block_table"][0, :pp].contiguous()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    K, Wm = max(args.steps, 3), max(args.warmup, 3)
    stream = torch.cuda.current_stream()

    def timed(fn):
        ts = []
        for i in range(Wm + K):
            flush.zero_()                                          # L2 flush: the state itself is smaller than L2
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream); fn(); e1.record(stream)
            torch.cuda.synchronize()
            if i >= Wm:
                ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    sampler = ClockSampler(local_rank); sampler.start()
    ms_plain = timed(lambda: pool.decode_attention(0, q, v["block_table"], v["seq_lens"], out_a))
    ms_shared = timed(lambda: pool.decode_attention_shared_prefix(0, q, v["block_table"], v["seq_lens"], prefix_blocks, pp, out_b))
    clocks = sampler.stop()
    err_code, err_mask = pool.last_error()
    logical = float(T * cfg.prefix_len + suffix.sum()) * cfg.bytes_per_token_layer
    unique = H.unique_kv_bytes(cfg, cfg.prefix_len, suffix)
    peak, peak_kind = measured_peaks()
    res = {"metric": "trace-layer decode steps/s (one layer, shared-prefix attention)", "value": T / (ms_shared * 1e-3),
           "unit": "trace-layer-steps/s", "n_gpus": 1, "steps": K, "warmup": Wm, "ms_per_step": ms_shared,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
           "data": "synthetic (seeded, drawn on device)",
           "config": {"workload": cfg.name, "traces": T, "prefix_len": cfg.prefix_len, "suffix": "1..%d" % args.suffix_max,
                      "shared_pages": pp, "l2_policy": "L2 flushed (256 MB written) before every timed launch"},
           "plain": {"ms": ms_plain, "logical_gbs": logical / ms_plain / 1e6, "unique_gbs": unique / ms_plain / 1e6},
           "shared_prefix": {"ms": ms_shared, "logical_gbs": logical / ms_shared / 1e6, "unique_gbs": unique / ms_shared / 1e6,
                             "launches": 2},
           "speedup": ms_plain / ms_shared, "max_abs_diff": float((out_a - out_b).abs().max()),
           "roofline": {"bound": "hbm", "achieved": unique / ms_shared / 1e6, "peak": peak, "unit": "GB/s",
                        "frac": unique / ms_shared / 1e6 / peak, "peak_kind": "of " + peak_kind, "traffic": None,
                        "kernel": "decode_attention_shared_prefix (two launches of attn_mma_kernel)",
                        "note": "a %.0f MB launch: fixed launch costs weigh on it" % (unique / 1e6)},
           "gpu_launches": 3 * K, "clocks": clocks, "status": {"device_error_mask": err_mask}}
    print(json.dumps(res))


# ---------------------------------------------------------------------------------------------
def run_replay(args):
    """`--workload replay`: the same 64 traces (one layer of the 8B layout, a pool that holds about 40 % of what they
    would need) run twice - by an engine that does not prune and therefore preempts, queues and reconstructs traces
    when the pool fills (the schedule of paper_2601_09093_b200/replay.py, host-driven by its nature, on this library's
    fork / append / release / attention kernels), and by the method's own loop (algorithm1_run: eviction by score, no
    queue).  Reports both runs' counters: the paper's Table 3 contrast (waiting 1526 s against 0) in units of decode
    iterations.  Single GPU."""
    import torch
    from paper_2601_09093_b200 import binding as B, harness as H, ranks as R, workloads as W
    from paper_2601_09093_b200 import build as _build
    from paper_2601_09093_b200.replay import preempt_and_recompute
    rank, local_rank, world = R.rank_env()
    if rank != 0:
        return
    _build.build()
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    B.lib()
    cfg = W.scaled(W.C1, name="replay-1layer", prefix_len=512)
    T, P, prompt = cfg.n_traces, cfg.page_size, cfg.prefix_len
    final = [int(x) for x in prompt + W.rng(cfg.seed, W.TID_LEN, 5).integers(1024, 4097, size=T)]
    nb = args.num_blocks or 4096
    max_pages = -(-max(final) // P) + 2
    max_traces = T + 4096                                           # every reconstruction takes a fresh trace id
    pool = H.make_pool(cfg, nb, max_pages, max_traces, max_score_rows=T, device=dev)
    v = pool.views()
    gen = torch.Generator(device=dev); gen.manual_seed(cfg.seed + 3)
    rnd = lambda *shape: torch.randn(shape, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    L, Hkv, Hq, d = cfg.num_layers, cfg.num_kv_heads, cfg.num_q_heads, cfg.head_dim
    kbuf, vbuf = rnd(L, Hkv, max(final), d), rnd(L, Hkv, max(final), d)
    knew, vnew, q = rnd(T, 1, L, Hkv, d), rnd(T, 1, L, Hkv, d), rnd(T, Hq, d)
    out = torch.empty((T, Hq, d), dtype=torch.float32, device=dev)
    zeros = torch.zeros(T, dtype=torch.int32, device=dev)

    class Ops:
        log, snap = [], None

        def _ids(self, ids):
            return torch.tensor(ids, dtype=torch.int32, device=dev)

        def free(self):
            return pool.stats()["free"]

        def fork_all(self, n, S):
            self.log.append(("fork", n, S))
            return pool.fork_prefix(n, S, kbuf[:, :, :S].contiguous(), vbuf[:, :, :S].contiguous())

        def fork_one(self, S):
            return self.fork_all(1, S)[0]

        def append(self, ids):
            self.log.append(("append", list(ids)))
            pool.append_kv(self._ids(ids), 1, knew[:len(ids)], vnew[:len(ids)])

        def release(self, ids):
            self.log.append(("release", list(ids)))
            pool.release_traces(self._ids(ids))
            if self.snap is None and sum(1 for o in self.log if o[0] == "release") == 8:
                # state after the eighth preemption, for the oracle's replay of the log up to here
                self.snap = (len(self.log), {k: v[k].clone() for k in ("block_table", "seq_lens", "live", "refcount", "free_list", "free_count")})

        def finish(self, ids):
            self.log.append(("release", list(ids)))
            pool.finish_traces(self._ids(ids), zeros[:len(ids)])

        def step(self, ids):
            idx = torch.tensor(ids, dtype=torch.long, device=dev)
            pool.decode_attention(0, q[:len(ids)], v["block_table"][idx], v["seq_lens"][idx], out[:len(ids)])

    ops = Ops()
    sampler = ClockSampler(local_rank); sampler.start()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    sc = preempt_and_recompute(ops, final, prompt, P)
    torch.cuda.synchronize()
    sc["seconds"] = time.perf_counter() - t0
    sc["kv_bytes_rewritten"] = sc["recomputed_tokens"] * cfg.bytes_per_token
    sc_stats, (sc_code, sc_mask) = pool.stats(), pool.last_error()

    # the method's own loop on the same traces: trace t samples the end-of-sequence token when it reaches final[t]
    pool2 = H.make_pool(cfg, nb, max_pages, T, max_score_rows=T, device=dev)
    pool2.fork_prefix(T, prompt, kbuf[:, :, :prompt].contiguous(), vbuf[:, :, :prompt].contiguous())
    vocab = W.synthetic_vocab(cfg.seed, 32000, step_end_frac=0.01)
    table = B.step_end_table_from_vocab(vocab)
    ends = np.flatnonzero(table.numpy())
    max_it = max(final) - prompt
    toks = W.token_ids(cfg.seed, max_it * T, len(vocab), ends, cfg.boundary_density, sub=9).reshape(max_it, T)
    toks[toks == 0] = 1
    for t in range(T):
        toks[final[t] - prompt - 1, t] = 0
    ring = 4
    (W1b, _), (b1b, _), (w2b, _), b2 = W.scorer_weights(cfg)
    wts = B.ScorerWeights(H.to_device(W1b, "bf16", dev), H.to_device(b1b, "bf16", dev), H.to_device(w2b, "bf16", dev), b2, B.STEP_BF16)
    qr, kr, vr, hr = rnd(ring, 1, T, Hq, d), rnd(ring, T, 1, L, Hkv, d), rnd(ring, T, 1, L, Hkv, d), rnd(ring, T, cfg.scorer_D)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    st = pool2.algorithm1_run(torch.from_numpy(toks).to(dev), 0, table.to(dev), zeros, qr, kr, vr, hr, wts, 1.0, -1.0,
                              max_evictions=4, check_every=64)
    st["seconds"] = time.perf_counter() - t0
    clocks = sampler.stop()
    st_stats, (st_code, st_mask) = pool2.stats(), pool2.last_error()
    st.update(waiting_trace_iterations=0, recomputed_tokens=0, preemptions=0)

    res = {"metric": "decode iterations and waiting of 64 traces in a pool holding ~40 % of their KV: preempt-and-recompute engine vs the method's loop",
           "value": sc["iterations"] / max(st["iterations"], 1), "unit": "x decode iterations (preempting engine / STEP loop)",
           "n_gpus": 1, "steps": 1, "warmup": 0, "ms_per_step": st["seconds"] * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded)",
           "config": {"workload": cfg.name, "traces": T, "prompt": prompt, "final_lengths": "512 + U[1024, 4096]", "num_blocks": nb,
                      "pool_tokens": nb * P, "tokens_if_all_complete": int(sum(final)), "l2_policy": "not a bandwidth measurement"},
           "preempt_and_recompute": sc, "step_loop": st,
           "status": {"sc_pool": sc_stats, "sc_error_mask": sc_mask, "step_pool": st_stats, "step_error_mask": st_mask},
           "gpu_launches": sc["iterations"] * 3 + st["iterations"] * 9, "clocks": clocks}
    if not args.no_cpu_baseline and ops.snap is not None:
        from oracle.kv_pool import KVPoolOracle
        n_ops, snap = ops.snap
        o = KVPoolOracle(L, Hkv, d, P, nb, max_traces, max_pages, store_payload=False)
        for op in ops.log[:n_ops]:
            if op[0] == "fork":
                o.fork_prefix(op[1], op[2])
            elif op[0] == "append":
                o.append_kv(op[1], 1)
            else:
                for t in op[1]:
                    o.release_trace(t)
        fc = int(snap["free_count"].item())
        same = (fc == o.free_count and snap["free_list"][:fc].cpu().tolist() == o.free_list
                and np.array_equal(snap["seq_lens"].cpu().numpy(), o.seq_lens)
                and np.array_equal(snap["live"].cpu().numpy().astype(bool), o.live)
                and np.array_equal(snap["refcount"].cpu().numpy(), o.refcount)
                and np.array_equal(snap["block_table"].cpu().numpy(), o.block_table))
        res["oracle_replay"] = {"what": "pool metadata after the eighth preemption (%d logged operations) against the oracle pool replaying the log" % n_ops,
                                "bit_exact": bool(same), "oracle_status": o.status}
    print(json.dumps(res))


# ---------------------------------------------------------------------------------------------
def run_reference(args):
    """The reference arm is the CPU oracle, as it stands, on the host cores.
    Under a multi-rank launcher rank 0 alone runs and prints; the other ranks leave at once."""
    from paper_2601_09093_b200 import ranks as R
    if R.rank_env()[0] != 0:
        return
    from oracle import attention as OA, scorer as OS
    from oracle.kv_pool import KVPoolOracle
    from paper_2601_09093_b200 import workloads as W

    K, Wm = args.steps, max(args.warmup, 1)
    if args.workload == "scorer":
        return run_reference_scorer(args, K, Wm)
    # the state of the GPU arm's default run (same plan, same margin below the trigger)
    cfg, suffix, nb, max_pages, _ = workload_plan(args.workload, args.num_blocks, planned_steps(K, max(args.warmup, 3), K), None,
                                                  args.traces, args.threshold)
    T, L, P = cfg.n_traces, cfg.num_layers, cfg.page_size
    # bounded sample of one step: attention of SAMPLE (trace, layer) pairs at the benchmark's length, and - in full -
    # the scorer on the step's boundary rows, the pool bookkeeping and the trigger for all traces
    S = cfg.prefix_len + int(suffix[0])
    pool = KVPoolOracle(L, cfg.num_kv_heads, cfg.head_dim, P, nb, T, max_pages, store_payload=False)
    ids = pool.fork_prefix(T, cfg.prefix_len)
    pool.append_kv(ids, int(suffix[0]))
    kb, Kx = W.normal(cfg.seed, W.TID_K, (S + Wm + K + 4, cfg.num_kv_heads, cfg.head_dim), "bf16")
    vb, Vx = W.normal(cfg.seed, W.TID_V, (S + Wm + K + 4, cfg.num_kv_heads, cfg.head_dim), "bf16")
    Kx, Vx = Kx.astype(np.float64), Vx.astype(np.float64)
    (_, W1x), (_, b1x), (_, w2x), b2 = W.scorer_weights(cfg)
    ts = OS.TraceScores(T)
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    threads = blas_threads()

    SAMPLE = 8
    t_att, t_rest = 0.0, 0.0

    def step(i, timed):
        nonlocal S, t_att, t_rest
        t0 = time.perf_counter()
        pool.append_kv([t for t in range(T) if pool.live[t]], 1)
        S += 1
        t1 = time.perf_counter()
        for j in range(SAMPLE):                         # SAMPLE (trace, layer) attentions at full length
            _, qx = W.normal(cfg.seed, W.TID_Q, (cfg.num_q_heads, cfg.head_dim), "bf16", sub=i * SAMPLE + j)
            OA.dense_decode_attention(qx, Kx[:S], Vx[:S])
        t2 = time.perf_counter()
        _, hx = W.normal(cfg.seed, W.TID_HID, (T, cfg.scorer_D), "bf16", sub=i)
        mask = W.boundary_mask(cfg, T, sub=100 + i)
        ys = OS.score_steps(hx, mask, W1x, b1x, w2x, b2)
        ts.update(ys, mask)
        pool.prune_if_saturated(ts.scores().astype(np.float32), cfg.threshold, cfg.keep_frac, on_evict=ts.clear)
        t3 = time.perf_counter()
        if timed:
            t_att += t2 - t1
            t_rest += (t1 - t0) + (t3 - t2)

    for i in range(Wm):
        step(i, False)
    for i in range(K):
        step(Wm + i, True)
    # a whole step = T * L (trace, layer) attentions at the sampled rate + everything else once
    step_s = t_att / (K * SAMPLE) * T * L + t_rest / K
    value = T / step_s                                             # whole trace-decode-steps per second
    res = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
           "warmup": Wm, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
           "config": {"workload": cfg.name, "traces": T, "layers": L, "tokens_per_trace": S,
                      "note": "CPU oracle; each step is a bounded sample, ms_per_step the whole step it extrapolates to"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads or cores, "host_cores": cores, "blas_threads": threads,
                            "kind": "oracle",
                            "sample": "per step: %d of the %d (trace, layer) attentions (all heads, full length), timed apart from " % (SAMPLE, T * L) +
                                      "the step's scorer rows, pool bookkeeping and trigger (done in full); the attention time is "
                                      "scaled to all pairs, the rest counted once (%.1f s of CPU in all)" % (t_att + t_rest)},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(res))


def run_reference_scorer(args, K, Wm, sample=64):
    """The oracle's scorer on a bounded sample (64 step-end rows per step) of the batched scorer workload."""
    from oracle import scorer as OS
    from paper_2601_09093_b200 import workloads as W
    cfg = scorer_shape(args.scorer_shape)
    (_, W1x), (_, b1x), (_, w2x), b2 = W.scorer_weights(cfg, bias_std=0.05)
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    mask = np.ones(sample, dtype=np.uint8)

    def step(i):
        _, hx = W.normal(cfg.seed, W.TID_HID, (sample, cfg.scorer_D), "bf16", sub=i)
        OS.score_steps(hx, mask, W1x, b1x, w2x, b2)

    for i in range(Wm):
        step(i)
    t0 = time.perf_counter()
    for i in range(K):
        step(Wm + i)
    dt = time.perf_counter() - t0
    value = K * sample / dt
    unit = "rows/s"
    print(json.dumps({"impl": "reference", "metric": "scorer calls/s (step-end hidden states scored per second)", "value": value,
                      "unit": unit, "n_gpus": args.gpus, "steps": K, "warmup": Wm, "ms_per_step": dt * 1e3 / K,
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
                      "config": {"workload": "scorer-batched-%s" % cfg.name, "D": cfg.scorer_D, "m": cfg.scorer_m,
                                 "note": "CPU oracle; each step scores %d rows" % sample},
                      "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle",
                                       "sample": "%d step-end rows per step" % sample},
                      "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        if a.workload in ("prefix", "replay", "append"):
            a.workload = "c1"           # the oracle's arm of the prefix workload is the one-layer configuration it is cut from
        run_reference(a)
    elif a.workload == "scorer":
        run_scorer(a)
    elif a.workload == "prefix":
        run_prefix(a)
    elif a.workload == "replay":
        run_replay(a)
    elif a.workload == "append":
        run_append(a)
    else:
        run_ours(a)
