"""ctypes binding of libstep.so - argument marshalling only.

Function names mirror the C header (include/step.h).  PyTorch is used for device memory and
streams; every step of the hot path runs in the library's CUDA kernels.  There is no CPU
fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstep.so")

STEP_OK = 0
STATUS_NAMES = {0: "STEP_OK", 1: "STEP_ERR_INVALID_ARG", 2: "STEP_ERR_NO_BLOCKS", 3: "STEP_ERR_BAD_TRACE",
                4: "STEP_ERR_CAPACITY", 5: "STEP_ERR_CUDA", 6: "STEP_ERR_TIMEOUT", 7: "STEP_ERR_BAD_BLOCK"}
STEP_BF16, STEP_FP32 = 0, 1
_TORCH_DTYPE = {STEP_BF16: torch.bfloat16, STEP_FP32: torch.float32}


class StepError(RuntimeError):
    def __init__(self, fn, code):
        super().__init__(f"{fn} failed: {STATUS_NAMES.get(code, code)}")
        self.code = code


class kv_pool_config(C.Structure):
    _fields_ = [("num_layers", C.c_int), ("num_q_heads", C.c_int), ("num_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("page_size", C.c_int), ("num_blocks", C.c_int),
                ("max_traces", C.c_int), ("max_pages_per_trace", C.c_int), ("dtype", C.c_int),
                ("max_score_rows", C.c_int), ("unscored_score", C.c_float),
                ("kv_storage", C.c_void_p), ("kv_bytes", C.c_size_t),
                ("meta_storage", C.c_void_p), ("meta_bytes", C.c_size_t)]


class scorer_weights(C.Structure):
    _fields_ = [("W1", C.c_void_p), ("b1", C.c_void_p), ("w2", C.c_void_p), ("b2", C.c_float),
                ("D", C.c_int), ("m", C.c_int), ("dtype", C.c_int)]


class step_iteration(C.Structure):
    _fields_ = [("n_traces", C.c_int), ("token_ids", C.c_void_p), ("eos_token", C.c_int),
                ("step_end_table", C.c_void_p), ("vocab", C.c_int), ("answers", C.c_void_p),
                ("n_layers_attention", C.c_int), ("q", C.c_void_p), ("k_new", C.c_void_p), ("v_new", C.c_void_p),
                ("hidden", C.c_void_p), ("attn_out", C.c_void_p), ("step_scores_out", C.c_void_p),
                ("boundary_mask_out", C.c_void_p), ("trace_scores_out", C.c_void_p), ("scorer", C.POINTER(scorer_weights)),
                ("threshold", C.c_float), ("keep_frac", C.c_float), ("max_evictions", C.c_int),
                ("pruned_ids_out", C.c_void_p), ("n_pruned_out", C.c_void_p)]


class step_run_args(C.Structure):
    _fields_ = [("n_traces", C.c_int), ("max_iterations", C.c_int), ("token_ids", C.c_void_p), ("eos_token", C.c_int),
                ("step_end_table", C.c_void_p), ("vocab", C.c_int), ("answers", C.c_void_p), ("ring", C.c_int),
                ("n_layers_attention", C.c_int), ("q", C.c_void_p), ("k_new", C.c_void_p), ("v_new", C.c_void_p),
                ("hidden", C.c_void_p), ("attn_out", C.c_void_p), ("step_scores_out", C.c_void_p),
                ("scorer", C.POINTER(scorer_weights)), ("threshold", C.c_float), ("keep_frac", C.c_float),
                ("max_evictions", C.c_int), ("check_every", C.c_int), ("score_history", C.c_void_p),
                ("use_graphs", C.c_int)]


class step_run_result(C.Structure):
    _fields_ = [("iterations", C.c_int), ("answer", C.c_int), ("answer_weight", C.c_float),
                ("n_finished", C.c_int), ("n_evicted", C.c_int), ("live_left", C.c_int)]


class scorer_train_hyper(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("pos_weight", C.c_float), ("step", C.c_int)]


_lib = None


def lib():
    """Loads libstep.so (built by paper_2601_09093_b200.build); raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2601_09093_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, ip, i = C.c_void_p, C.POINTER(C.c_int), C.c_int
    L.step_version.restype = C.c_char_p
    L.kv_pool_required_bytes.argtypes = [C.POINTER(kv_pool_config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.kv_pool_create.argtypes = [C.POINTER(kv_pool_config), C.POINTER(vp)]
    L.kv_pool_destroy.argtypes = [vp]
    L.kv_pool_reset.argtypes = [vp, vp]
    L.kv_pool_fork_prefix.argtypes = [vp, i, i, vp, vp, ip, vp]
    L.append_kv.argtypes = [vp, vp, i, i, vp, vp, vp]
    L.decode_attention.argtypes = [vp, i, vp, vp, vp, i, vp, vp]
    L.decode_attention_static.argtypes = [vp, i, vp, vp, vp, i, vp, vp]
    L.decode_attention_dependent.argtypes = [vp, i, vp, vp, vp, i, vp, vp]
    L.step_read_stream_probe.argtypes = [vp, C.c_size_t, i, i, vp, vp]
    L.decode_attention_layers.argtypes = [vp, i, i, vp, vp, vp, i, vp, vp]
    L.decode_attention_shared_prefix.argtypes = [vp, i, vp, vp, vp, i, vp, i, vp, vp]
    L.score_steps.argtypes = [vp, vp, vp, vp, i, C.POINTER(scorer_weights), vp, vp]
    L.score_steps_tokens.argtypes = [vp, vp, vp, vp, i, vp, i, C.POINTER(scorer_weights), vp, vp, vp]
    L.detect_step_ends.argtypes = [vp, vp, i, vp, i, vp, vp]
    L.step_end_table_from_vocab.argtypes = [C.POINTER(C.c_char_p), ip, i, vp]
    L.prune_if_saturated.argtypes = [vp, vp, C.c_float, C.c_float, vp, vp, vp]
    L.kv_pool_release_traces.argtypes = [vp, vp, i, vp]
    L.kv_pool_stats.argtypes = [vp, ip, ip, ip, ip, vp]
    L.kv_pool_device_views.argtypes = [vp] + [C.POINTER(vp)] * 7
    L.kv_pool_score_views.argtypes = [vp] + [C.POINTER(vp)] * 2
    L.kv_pool_last_error.argtypes = [vp, C.POINTER(C.c_uint), vp]
    L.kv_pool_read_kv.argtypes = [vp, i, i, vp, i, vp, vp, vp]
    L.kv_pool_set_attention_config.argtypes = [vp, i, i]
    L.kv_pool_set_attention_balance.argtypes = [vp, i, i]
    L.kv_pool_set_wait_limit_ns.argtypes = [vp, C.c_ulonglong]
    L.scorer_train_workspace_bytes.argtypes = [i, i, i]
    L.scorer_train_workspace_bytes.restype = C.c_size_t
    L.scorer_train_step.argtypes = [vp, i, vp, i, vp, vp, vp, vp, i, i, vp, vp, C.POINTER(scorer_train_hyper), vp, C.c_size_t, vp, vp]
    L.kv_pool_finish_traces.argtypes = [vp, vp, vp, i, vp]
    L.weighted_vote.argtypes = [vp, vp, vp, vp, vp]
    L.kv_pool_vote_views.argtypes = [vp] + [C.POINTER(vp)] * 3
    L.algorithm1_iteration.argtypes = [vp, C.POINTER(step_iteration), vp]
    L.algorithm1_run.argtypes = [vp, C.POINTER(step_run_args), C.POINTER(step_run_result), vp]
    L.kv_pool_set_scorer_config.argtypes = [vp, i, i]
    L.kv_pool_score_launch_info.argtypes = [vp, ip, ip, vp]
    _lib = L
    return L


def _check(fn, code):
    if code != STEP_OK:
        raise StepError(fn, code)


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def kv_pool_required_bytes(**geometry):
    cfg = kv_pool_config(**geometry)
    kb, mb = C.c_size_t(), C.c_size_t()
    _check("kv_pool_required_bytes", lib().kv_pool_required_bytes(C.byref(cfg), C.byref(kb), C.byref(mb)))
    return kb.value, mb.value


class KVPool:
    """Owns the torch tensors behind one step_pool and forwards the C calls."""

    def __init__(self, num_layers, num_q_heads, num_kv_heads, head_dim, page_size, num_blocks, max_traces,
                 max_pages_per_trace, dtype=STEP_BF16, max_score_rows=0, unscored_score=1.0, device="cuda:0"):
        self.geometry = dict(num_layers=num_layers, num_q_heads=num_q_heads, num_kv_heads=num_kv_heads,
                             head_dim=head_dim, page_size=page_size, num_blocks=num_blocks, max_traces=max_traces,
                             max_pages_per_trace=max_pages_per_trace, dtype=dtype, max_score_rows=max_score_rows,
                             unscored_score=unscored_score)
        self.dtype, self.torch_dtype = dtype, _TORCH_DTYPE[dtype]
        self.device = torch.device(device)
        kb, mb = kv_pool_required_bytes(**self.geometry)
        self.kv_bytes, self.meta_bytes = kb, mb
        with torch.cuda.device(self.device):
            self.kv_storage = torch.empty(kb, dtype=torch.uint8, device=self.device)
            self.meta_storage = torch.empty(mb, dtype=torch.uint8, device=self.device)
            cfg = kv_pool_config(kv_storage=self.kv_storage.data_ptr(), kv_bytes=kb,
                                 meta_storage=self.meta_storage.data_ptr(), meta_bytes=mb, **self.geometry)
            h = C.c_void_p()
            _check("kv_pool_create", lib().kv_pool_create(C.byref(cfg), C.byref(h)))
        self.handle = h
        for k, v in self.geometry.items():
            setattr(self, k, v)
        self._views = None
        self.pruned_ids = torch.empty(max_traces, dtype=torch.int32, device=self.device)
        self.n_pruned = torch.zeros(1, dtype=torch.int32, device=self.device)

    def close(self):
        if self.handle is not None:
            lib().kv_pool_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- views into meta_storage as torch tensors (no copies)
    def _view(self, ptr, count, dtype):
        off = ptr - self.meta_storage.data_ptr()
        nbytes = count * torch.empty(0, dtype=dtype).element_size()
        return self.meta_storage[off:off + nbytes].view(dtype)

    def views(self):
        if self._views is None:
            p = [C.c_void_p() for _ in range(7)]
            _check("kv_pool_device_views", lib().kv_pool_device_views(self.handle, *[C.byref(x) for x in p]))
            q = [C.c_void_p() for _ in range(2)]
            _check("kv_pool_score_views", lib().kv_pool_score_views(self.handle, *[C.byref(x) for x in q]))
            T, NB, MP = self.max_traces, self.num_blocks, self.max_pages_per_trace
            self._views = dict(
                block_table=self._view(p[0].value, T * MP, torch.int32).view(T, MP),
                seq_lens=self._view(p[1].value, T, torch.int32),
                trace_scores=self._view(p[2].value, T, torch.float32),
                free_list=self._view(p[3].value, NB, torch.int32),
                free_count=self._view(p[4].value, 1, torch.int32),
                refcount=self._view(p[5].value, NB, torch.int32),
                live=self._view(p[6].value, T, torch.uint8),
                score_sum=self._view(q[0].value, T, torch.float32),
                score_cnt=self._view(q[1].value, T, torch.int32))
        return self._views

    # ---- the calls
    def reset(self, stream=None):
        _check("kv_pool_reset", lib().kv_pool_reset(self.handle, _stream(stream)))

    def fork_prefix(self, n_traces, prefix_len, k_prefix, v_prefix, stream=None):
        ids = (C.c_int * n_traces)()
        _check("kv_pool_fork_prefix", lib().kv_pool_fork_prefix(self.handle, n_traces, prefix_len, _ptr(k_prefix),
                                                                _ptr(v_prefix), ids, _stream(stream)))
        return [] if ids[0] < 0 else list(ids)           # a fork that failed on the device hands out no ids

    def append_kv(self, trace_ids, n_tokens, k_new, v_new, stream=None):
        _check("append_kv", lib().append_kv(self.handle, _ptr(trace_ids), trace_ids.numel(), n_tokens, _ptr(k_new),
                                            _ptr(v_new), _stream(stream)))

    def decode_attention(self, layer, q, block_table, seq_lens, out=None, stream=None):
        n = q.shape[0]
        if out is None:
            out = torch.empty((n, self.num_q_heads, self.head_dim), dtype=torch.float32, device=q.device)
        _check("decode_attention", lib().decode_attention(self.handle, layer, _ptr(q), _ptr(block_table), _ptr(seq_lens),
                                                          n, _ptr(out), _stream(stream)))
        return out

    def decode_attention_dependent(self, layer, q, block_table, seq_lens, out=None, stream=None):
        """decode_attention launched as a programmatic dependent of the kernel that precedes it in the stream (the one
        that writes q)."""
        n = q.shape[0]
        if out is None:
            out = torch.empty((n, self.num_q_heads, self.head_dim), dtype=torch.float32, device=q.device)
        _check("decode_attention_dependent", lib().decode_attention_dependent(self.handle, layer, _ptr(q), _ptr(block_table),
                                                                              _ptr(seq_lens), n, _ptr(out), _stream(stream)))
        return out

    def decode_attention_layers(self, layer0, q, block_table, seq_lens, out=None, stream=None):
        """q: [n_layers, n, Hq, d] -> out [n_layers, n, Hq, d] fp32: layers layer0 .. layer0 + n_layers - 1."""
        n_layers, n = q.shape[0], q.shape[1]
        if out is None:
            out = torch.empty((n_layers, n, self.num_q_heads, self.head_dim), dtype=torch.float32, device=q.device)
        _check("decode_attention_layers", lib().decode_attention_layers(self.handle, layer0, n_layers, _ptr(q), _ptr(block_table),
                                                                        _ptr(seq_lens), n, _ptr(out), _stream(stream)))
        return out

    def decode_attention_shared_prefix(self, layer, q, block_table, seq_lens, prefix_blocks, prefix_pages, out=None, stream=None):
        n = q.shape[0]
        if out is None:
            out = torch.empty((n, self.num_q_heads, self.head_dim), dtype=torch.float32, device=q.device)
        _check("decode_attention_shared_prefix", lib().decode_attention_shared_prefix(
            self.handle, layer, _ptr(q), _ptr(block_table), _ptr(seq_lens), n, _ptr(prefix_blocks), prefix_pages,
            _ptr(out), _stream(stream)))
        return out

    def decode_attention_static(self, layer, q, block_table, seq_lens, out, stream=None):
        """The allocation-free variant: `out` must be supplied by the caller; nothing is allocated."""
        _check("decode_attention_static", lib().decode_attention_static(self.handle, layer, _ptr(q), _ptr(block_table),
                                                                        _ptr(seq_lens), q.shape[0], _ptr(out), _stream(stream)))
        return out

    def score_steps(self, hidden, boundary_mask, row_trace, weights, step_scores_out=None, stream=None):
        M = hidden.shape[0]
        if step_scores_out is None:
            step_scores_out = torch.empty(M, dtype=torch.float32, device=hidden.device)
        _check("score_steps", lib().score_steps(self.handle, _ptr(hidden), _ptr(boundary_mask), _ptr(row_trace), M,
                                                C.byref(weights.struct), _ptr(step_scores_out), _stream(stream)))
        return step_scores_out

    def score_steps_tokens(self, hidden, token_ids, step_end_table, row_trace, weights, step_scores_out=None,
                           boundary_mask_out=None, stream=None):
        M = hidden.shape[0]
        if step_scores_out is None:
            step_scores_out = torch.empty(M, dtype=torch.float32, device=hidden.device)
        _check("score_steps_tokens", lib().score_steps_tokens(
            self.handle, _ptr(hidden), _ptr(token_ids), _ptr(step_end_table), step_end_table.numel(), _ptr(row_trace), M,
            C.byref(weights.struct), _ptr(step_scores_out), _ptr(boundary_mask_out), _stream(stream)))
        return step_scores_out

    def detect_step_ends(self, token_ids, step_end_table, boundary_mask_out=None, stream=None):
        M = token_ids.numel()
        if boundary_mask_out is None:
            boundary_mask_out = torch.empty(M, dtype=torch.uint8, device=token_ids.device)
        _check("detect_step_ends", lib().detect_step_ends(self.handle, _ptr(token_ids), M, _ptr(step_end_table),
                                                          step_end_table.numel(), _ptr(boundary_mask_out), _stream(stream)))
        return boundary_mask_out

    def prune_if_saturated(self, scores, threshold, keep_frac, stream=None):
        """Returns (pruned_ids, n_pruned) device tensors owned by the pool (no sync)."""
        _check("prune_if_saturated", lib().prune_if_saturated(self.handle, _ptr(scores), threshold, keep_frac,
                                                              _ptr(self.pruned_ids), _ptr(self.n_pruned), _stream(stream)))
        return self.pruned_ids, self.n_pruned

    def release_traces(self, trace_ids, stream=None):
        _check("kv_pool_release_traces", lib().kv_pool_release_traces(self.handle, _ptr(trace_ids), trace_ids.numel(),
                                                                      _stream(stream)))

    def stats(self, stream=None):
        u, f, t, l = C.c_int(), C.c_int(), C.c_int(), C.c_int()
        _check("kv_pool_stats", lib().kv_pool_stats(self.handle, C.byref(u), C.byref(f), C.byref(t), C.byref(l), _stream(stream)))
        return dict(used=u.value, free=f.value, total=t.value, live_traces=l.value)

    def last_error(self, stream=None):
        mask = C.c_uint()
        code = lib().kv_pool_last_error(self.handle, C.byref(mask), _stream(stream))
        return code, mask.value

    def read_kv(self, layer, kv_head, block_row, seq_len, stream=None):
        k = torch.empty((seq_len, self.head_dim), dtype=self.torch_dtype, device=self.device)
        v = torch.empty_like(k)
        _check("kv_pool_read_kv", lib().kv_pool_read_kv(self.handle, layer, kv_head, _ptr(block_row), seq_len, _ptr(k),
                                                        _ptr(v), _stream(stream)))
        return k, v

    # ---- Algorithm 1 as a loop
    def finish_traces(self, trace_ids, answers, stream=None):
        _check("kv_pool_finish_traces", lib().kv_pool_finish_traces(self.handle, _ptr(trace_ids), _ptr(answers),
                                                                    trace_ids.numel(), _stream(stream)))

    def weighted_vote(self, stream=None):
        """Returns device tensors (answer [1] int32, weight [1] float32, n_finished [1] int32); no sync."""
        a = torch.empty(1, dtype=torch.int32, device=self.device)
        w = torch.empty(1, dtype=torch.float32, device=self.device)
        n = torch.empty(1, dtype=torch.int32, device=self.device)
        _check("weighted_vote", lib().weighted_vote(self.handle, _ptr(a), _ptr(w), _ptr(n), _stream(stream)))
        return a, w, n

    def vote_views(self):
        p = [C.c_void_p() for _ in range(3)]
        _check("kv_pool_vote_views", lib().kv_pool_vote_views(self.handle, *[C.byref(x) for x in p]))
        T = self.max_traces
        return dict(final_score=self._view(p[0].value, T, torch.float32), answer=self._view(p[1].value, T, torch.int32),
                    finished=self._view(p[2].value, T, torch.uint8))

    def algorithm1_iteration(self, token_ids, eos_token, step_end_table, answers, q, k_new, v_new, hidden, weights,
                             threshold, keep_frac, max_evictions=1, attn_out=None, step_scores_out=None,
                             boundary_mask_out=None, trace_scores_out=None, pruned_ids_out=None, n_pruned_out=None,
                             stream=None):
        """One iteration of the loop for traces 0 .. n-1 (row i of every input is trace i); no sync.
        q: [layers, n, Hq, d] or None (no attention)."""
        n = token_ids.numel()
        La = 0 if q is None else q.shape[0]
        if La and attn_out is None:
            attn_out = torch.empty((La, n, self.num_q_heads, self.head_dim), dtype=torch.float32, device=self.device)
        if step_scores_out is None:
            step_scores_out = torch.empty(n, dtype=torch.float32, device=self.device)
        it = step_iteration(n_traces=n, token_ids=token_ids.data_ptr(), eos_token=eos_token,
                            step_end_table=step_end_table.data_ptr(), vocab=step_end_table.numel(),
                            answers=_ptr(answers).value, n_layers_attention=La, q=_ptr(q).value, k_new=k_new.data_ptr(),
                            v_new=v_new.data_ptr(), hidden=hidden.data_ptr(), attn_out=_ptr(attn_out).value,
                            step_scores_out=step_scores_out.data_ptr(), boundary_mask_out=_ptr(boundary_mask_out).value,
                            trace_scores_out=_ptr(trace_scores_out).value, scorer=C.pointer(weights.struct), threshold=threshold, keep_frac=keep_frac,
                            max_evictions=max_evictions, pruned_ids_out=_ptr(pruned_ids_out).value, n_pruned_out=_ptr(n_pruned_out).value)
        _check("algorithm1_iteration", lib().algorithm1_iteration(self.handle, C.byref(it), _stream(stream)))
        return attn_out, step_scores_out

    def algorithm1_run(self, token_ids, eos_token, step_end_table, answers, q, k_new, v_new, hidden, weights, threshold,
                       keep_frac, max_evictions=1, check_every=16, attn_out=None, score_history=None, stream=None,
                       use_graphs=False):
        """The whole loop.  token_ids: [max_iterations, n]; q: [ring, layers, n, Hq, d] or None;
        k_new, v_new: [ring, n, 1, L, Hkv, d]; hidden: [ring, n, D].  Returns the result as a dict (synchronises)."""
        max_it, n = token_ids.shape
        ring = k_new.shape[0]
        La = 0 if q is None else q.shape[1]
        if La and attn_out is None:
            attn_out = torch.empty((La, n, self.num_q_heads, self.head_dim), dtype=torch.float32, device=self.device)
        scores = torch.empty(n, dtype=torch.float32, device=self.device)
        a = step_run_args(n_traces=n, max_iterations=max_it, token_ids=token_ids.data_ptr(), eos_token=eos_token,
                          step_end_table=step_end_table.data_ptr(), vocab=step_end_table.numel(), answers=_ptr(answers).value,
                          ring=ring, n_layers_attention=La, q=_ptr(q).value, k_new=k_new.data_ptr(), v_new=v_new.data_ptr(),
                          hidden=hidden.data_ptr(), attn_out=_ptr(attn_out).value, step_scores_out=scores.data_ptr(),
                          scorer=C.pointer(weights.struct), threshold=threshold, keep_frac=keep_frac, max_evictions=max_evictions, check_every=check_every,
                          score_history=_ptr(score_history).value, use_graphs=int(bool(use_graphs)))
        r = step_run_result()
        _check("algorithm1_run", lib().algorithm1_run(self.handle, C.byref(a), C.byref(r), _stream(stream)))
        return {k: getattr(r, k) for k, _ in step_run_result._fields_}

    def set_attention_config(self, grid_ctas=0, fast_path=0):
        _check("kv_pool_set_attention_config", lib().kv_pool_set_attention_config(self.handle, grid_ctas, fast_path))

    def set_attention_balance(self, dynamic_sixteenths, min_chunk_pages=0):
        _check("kv_pool_set_attention_balance",
               lib().kv_pool_set_attention_balance(self.handle, dynamic_sixteenths, min_chunk_pages))

    def set_wait_limit_ns(self, ns):
        _check("kv_pool_set_wait_limit_ns", lib().kv_pool_set_wait_limit_ns(self.handle, ns))

    def set_scorer_config(self, mode=0, tc_min_rows=0):
        _check("kv_pool_set_scorer_config", lib().kv_pool_set_scorer_config(self.handle, mode, tc_min_rows))

    def score_launch_info(self, stream=None):
        n, u = C.c_int(), C.c_int()
        _check("kv_pool_score_launch_info", lib().kv_pool_score_launch_info(self.handle, C.byref(n), C.byref(u), _stream(stream)))
        return dict(n_rows=n.value, tc_units=u.value)


class ScorerTrainer:
    """fp32 scorer parameters, Adam moments and workspace on the device; step() forwards to scorer_train_step."""

    def __init__(self, W1, b1, w2, b2, batch, lr=1e-4, weight_decay=1e-5, pos_weight=1.0, beta1=0.9, beta2=0.999, eps=1e-8):
        self.W1, self.b1, self.w2 = (x.to(torch.float32, copy=True).contiguous() for x in (W1, b1, w2))   # owned copies
        self.b2 = torch.tensor([float(b2)], dtype=torch.float32, device=self.W1.device)
        self.m, self.D = self.W1.shape
        n = self.m * self.D + 2 * self.m + 1
        self.adam_m = torch.zeros(n, dtype=torch.float32, device=self.W1.device)
        self.adam_v = torch.zeros_like(self.adam_m)
        self.batch = batch
        self.ws_bytes = lib().scorer_train_workspace_bytes(batch, self.D, self.m)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.W1.device)
        self.loss = torch.zeros(1, dtype=torch.float32, device=self.W1.device)
        self.h = scorer_train_hyper(lr=lr, beta1=beta1, beta2=beta2, eps=eps, weight_decay=weight_decay,
                                    pos_weight=pos_weight, step=0)

    def step(self, hidden, labels, stream=None):
        """One update; returns the device tensor holding the loss before the update (no sync)."""
        assert hidden.shape == (self.batch, self.D) and labels.dtype == torch.float32
        self.h.step += 1
        dt = STEP_BF16 if hidden.dtype == torch.bfloat16 else STEP_FP32
        _check("scorer_train_step", lib().scorer_train_step(
            _ptr(hidden), dt, _ptr(labels), self.batch, _ptr(self.W1), _ptr(self.b1), _ptr(self.w2), _ptr(self.b2),
            self.D, self.m, _ptr(self.adam_m), _ptr(self.adam_v), C.byref(self.h), _ptr(self.ws), self.ws_bytes,
            _ptr(self.loss), _stream(stream)))
        return self.loss


def read_stream_probe(buf, n_launches, chained, err_flag, stream=None):
    """step_read_stream_probe over the bytes of `buf` (a contiguous device tensor); no sync."""
    _check("step_read_stream_probe", lib().step_read_stream_probe(_ptr(buf), buf.numel() * buf.element_size(), n_launches,
                                                                  int(bool(chained)), _ptr(err_flag), _stream(stream)))


def step_end_table_from_vocab(token_texts):
    """Host table (torch.uint8, [vocab]) marking the vocabulary entries whose text contains two newlines in a row.
    token_texts: a sequence of bytes objects (None = empty)."""
    n = len(token_texts)
    arr = (C.c_char_p * n)(*[t if t is not None else None for t in token_texts])
    lens = (C.c_int * n)(*[len(t) if t is not None else 0 for t in token_texts])
    out = torch.zeros(n, dtype=torch.uint8)
    _check("step_end_table_from_vocab", lib().step_end_table_from_vocab(arr, lens, n, C.c_void_p(out.data_ptr())))
    return out


class ScorerWeights:
    """Device tensors of the step scorer plus the C struct that points at them."""

    def __init__(self, W1, b1, w2, b2, dtype):
        self.W1, self.b1, self.w2, self.b2 = W1.contiguous(), b1.contiguous(), w2.contiguous(), float(b2)
        m, D = self.W1.shape
        self.struct = scorer_weights(W1=self.W1.data_ptr(), b1=self.b1.data_ptr(), w2=self.w2.data_ptr(),
                                     b2=self.b2, D=D, m=m, dtype=dtype)
