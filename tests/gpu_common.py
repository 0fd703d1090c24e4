"""Helpers for the GPU parity tests: drive the CUDA pool and the oracle pool with the same inputs."""
import numpy as np
import torch

from oracle.kv_pool import KVPoolOracle
from paper_2601_09093_b200 import binding as B
from paper_2601_09093_b200 import harness as H
from paper_2601_09093_b200 import workloads as W


class Twin:
    """A CUDA pool and an oracle pool fed identical seeded data."""

    def __init__(self, cfg: W.Config, num_blocks, max_pages, max_traces=None, shuffle=False, store_payload=True,
                 max_score_rows=0):
        self.cfg = cfg
        T = max_traces or cfg.n_traces
        self.gpu = H.make_pool(cfg, num_blocks, max_pages, T, max_score_rows=max_score_rows)
        self.ora = KVPoolOracle(cfg.num_layers, cfg.num_kv_heads, cfg.head_dim, cfg.page_size, num_blocks, T,
                                max_pages, store_payload=store_payload)
        if shuffle:
            H.shuffle_free_list(self.gpu, cfg.seed)
            self.ora.free_list = [int(x) for x in W.block_permutation(cfg.seed, num_blocks)]
        self.sub = 0

    def _draw(self, tid, shape):
        self.sub += 1
        return W.normal(self.cfg.seed, tid, shape, self.cfg.dtype, sub=self.sub)

    def fork(self, n, prefix_len):
        c = self.cfg
        shape = (c.num_layers, c.num_kv_heads, prefix_len, c.head_dim)
        kb, kx = self._draw(W.TID_KPRE, shape)
        vb, vx = self._draw(W.TID_VPRE, shape)
        ids = self.gpu.fork_prefix(n, prefix_len, H.to_device(kb, c.dtype), H.to_device(vb, c.dtype))
        oids = self.ora.fork_prefix(n, prefix_len, kx, vx)
        return ids, oids

    def append(self, ids, n_tokens):
        c = self.cfg
        shape = (len(ids), n_tokens, c.num_layers, c.num_kv_heads, c.head_dim)
        if self.ora.store_payload:
            kb, kx = self._draw(W.TID_KNEW, shape)
            vb, vx = self._draw(W.TID_VNEW, shape)
            kd, vd = H.to_device(kb, c.dtype), H.to_device(vb, c.dtype)
        else:
            kx = vx = None
            kd = torch.zeros(shape, dtype=self.gpu.torch_dtype, device=self.gpu.device)
            vd = kd
        self.gpu.append_kv(torch.tensor(list(ids), dtype=torch.int32, device=self.gpu.device), n_tokens, kd, vd)
        return self.ora.append_kv(list(ids), n_tokens, kx, vx)

    def assert_meta_equal(self):
        v = self.gpu.views()
        torch.cuda.synchronize()
        o = self.ora
        fc = int(v["free_count"].item())
        assert fc == o.free_count, (fc, o.free_count)
        assert v["free_list"][:fc].cpu().tolist() == o.free_list, "free list differs"
        np.testing.assert_array_equal(v["seq_lens"].cpu().numpy(), o.seq_lens)
        np.testing.assert_array_equal(v["live"].cpu().numpy().astype(bool), o.live)
        np.testing.assert_array_equal(v["refcount"].cpu().numpy(), o.refcount)
        np.testing.assert_array_equal(v["block_table"].cpu().numpy(), o.block_table)
        o.check_invariants()

    def status(self):
        code, mask = self.gpu.last_error()
        omask = self.ora.status
        self.ora.status = 0
        return mask, omask


def exact_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def attention_errors(got: np.ndarray, want: np.ndarray):
    err = np.abs(got.astype(np.float64) - want)
    return float(err.max()) if err.size else 0.0, float(err.mean()) if err.size else 0.0
