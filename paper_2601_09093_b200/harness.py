"""Device-side workload construction shared by the GPU tests, the smoke check and bench.py.

Only plumbing lives here: moving seeded inputs (workloads.py) to the GPU and driving the
library calls that build a KV pool of the requested shape.  No arithmetic of the method.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import workloads as W


def to_device(bits_or_f32: np.ndarray, dtype: str, device="cuda:0") -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor; float32 stays float32."""
    if dtype == "bf16":
        return torch.from_numpy(np.ascontiguousarray(bits_or_f32).view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(bits_or_f32, dtype=np.float32)).to(device)


def step_dtype(cfg: W.Config) -> int:
    return B.STEP_BF16 if cfg.dtype == "bf16" else B.STEP_FP32


def make_pool(cfg: W.Config, num_blocks: int, max_pages: int, max_traces=None, max_score_rows=0,
              device="cuda:0") -> B.KVPool:
    return B.KVPool(cfg.num_layers, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.page_size, num_blocks,
                    max_traces or cfg.n_traces, max_pages, dtype=step_dtype(cfg), max_score_rows=max_score_rows,
                    device=device)


def ragged_append_plan(lengths):
    """Appends that give trace i exactly lengths[i] new tokens using bulk calls.

    Yields (trace_index_array, n_tokens): traces sorted by length; call k appends the k-th
    length increment to every trace that still needs tokens.
    """
    order = np.argsort(lengths, kind="stable")
    done = 0
    for pos, idx in enumerate(order):
        inc = int(lengths[idx]) - done
        if inc > 0:
            yield np.sort(order[pos:]).astype(np.int32), inc
            done += inc


def fill_random_device(pool: B.KVPool, cfg: W.Config, lengths, seed: int, chunk_tokens=2048, log=None):
    """Forks cfg.n_traces traces from a random prompt and grows trace i by lengths[i] tokens.

    K/V values are N(0,1) drawn ON THE DEVICE from a seeded torch generator (the pools of the large
    configurations are far too big to draw on the host); parity tests read the stored rows back
    through kv_pool_read_kv and hand those bytes to the oracle.  `log`, if given, receives one
    (trace id list, n_tokens) entry per append_kv call, in call order.
    """
    dev = pool.device
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    L, Hkv, d = cfg.num_layers, cfg.num_kv_heads, cfg.head_dim
    tdt = pool.torch_dtype
    kp = torch.randn((L, Hkv, cfg.prefix_len, d), generator=gen, device=dev, dtype=torch.float32).to(tdt)
    vp = torch.randn((L, Hkv, cfg.prefix_len, d), generator=gen, device=dev, dtype=torch.float32).to(tdt)
    ids = pool.fork_prefix(len(lengths), cfg.prefix_len, kp, vp)
    ids_np = np.asarray(ids, dtype=np.int32)
    for sel, inc in ragged_append_plan(lengths):
        tid = torch.from_numpy(ids_np[sel]).to(dev)
        left = inc
        while left > 0:
            c = min(left, chunk_tokens)
            kn = torch.randn((len(sel), c, L, Hkv, d), generator=gen, device=dev, dtype=torch.float32).to(tdt)
            vn = torch.randn((len(sel), c, L, Hkv, d), generator=gen, device=dev, dtype=torch.float32).to(tdt)
            pool.append_kv(tid, c, kn, vn)
            if log is not None:
                log.append((ids_np[sel].tolist(), c))
            left -= c
    return ids


def shuffle_free_list(pool: B.KVPool, seed: int):
    """Scatters future allocations across the pool: permutes the (all-free) free list."""
    perm = W.block_permutation(seed, pool.num_blocks)
    pool.views()["free_list"].copy_(torch.from_numpy(perm).to(pool.device))


def unique_kv_bytes(cfg: W.Config, prefix_len: int, suffix_lens) -> int:
    """KV bytes one layer-call must read when the shared prompt is counted once."""
    return int((prefix_len + int(np.sum(suffix_lens))) * cfg.bytes_per_token_layer)
