"""Thin ctypes binding of libfspad.so: argument marshalling only.

Every function takes torch tensors (device memory, streams), checks dtype,
shape and contiguity, and forwards raw pointers to the C ABI declared in
`include/fspad.h`.  No step of the verify path is computed here, and there is
no fallback: if the library has not been built the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libfspad.so")
_lib = None

EXPORTS = ["fspad_create", "fspad_destroy", "fspad_status", "fspad_strerror", "fspad_launch_count",
           "fspad_tree_attn", "fspad_tree_accept", "fspad_accept_stats", "fspad_kv_compact",
           "fspad_tree_attn_paged", "fspad_kv_compact_paged", "fspad_kv_append", "fspad_lm_head_stats", "fspad_lm_head_accept", "fspad_feature_sampler", "fspad_feature_sampler_workspace_bytes", "fspad_verify_step", "fspad_verify_step_host", "fspad_selftest_wait_timeout", "fspad_accept_stats_noalloc", "fspad_tree_build", "fspad_draft_expand"]


class FspadConfig(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int), ("n_kv_heads", ctypes.c_int), ("head_dim", ctypes.c_int),
                ("max_nodes", ctypes.c_int), ("vocab", ctypes.c_int), ("n_layers", ctypes.c_int),
                ("max_len", ctypes.c_int), ("max_batch", ctypes.c_int), ("softmax_scale", ctypes.c_float)]


class FspadError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, strerror(code), code))


def load():
    """Open libfspad.so (built in-tree by `python -m paper_2408_15562_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libfspad.so is missing: build it with `python -m paper_2408_15562_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    lib.fspad_create.argtypes = [ctypes.POINTER(FspadConfig), ctypes.POINTER(vp)]
    lib.fspad_destroy.argtypes = [vp]
    lib.fspad_destroy.restype = None
    lib.fspad_status.argtypes = [vp, vp]
    lib.fspad_strerror.argtypes = [ci]
    lib.fspad_strerror.restype = ctypes.c_char_p
    lib.fspad_launch_count.argtypes = [vp]
    lib.fspad_launch_count.restype = ctypes.c_longlong
    lib.fspad_tree_attn.argtypes = [vp] * 8 + [ci, ci, vp, vp]
    lib.fspad_tree_accept.argtypes = [vp] * 7 + [ci, ci, vp, vp, vp, vp]
    lib.fspad_accept_stats.argtypes = [vp, vp, vp, ci, ci, vp, vp, vp, vp]
    lib.fspad_kv_compact.argtypes = [vp, vp, vp, vp, vp, ci, vp, vp]
    lib.fspad_accept_stats_noalloc.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, vp]
    lib.fspad_lm_head_stats.argtypes = [vp, vp, vp, ci, ci, ci, vp, vp, vp, vp, vp, vp]
    lib.fspad_lm_head_accept.argtypes = [vp, vp, vp, ci, vp, vp, vp, vp, vp, ci, ci, vp, vp, vp, vp, vp]
    lib.fspad_feature_sampler_workspace_bytes.argtypes = [ci, ci, ci]
    lib.fspad_feature_sampler_workspace_bytes.restype = ctypes.c_size_t
    lib.fspad_feature_sampler.argtypes = [vp] * 6 + [ci, ci, ci, vp, vp, vp, ctypes.c_size_t, vp]
    lib.fspad_tree_attn_paged.argtypes = [vp, vp, vp, vp, vp, ci, ci, vp, vp, vp, vp, ci, ci, vp, vp]
    lib.fspad_kv_append.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, vp, vp]
    lib.fspad_kv_compact_paged.argtypes = [vp, vp, vp, ci, ci, vp, vp, vp, ci, vp, vp]
    lib.fspad_selftest_wait_timeout.argtypes = [vp, ci, vp]
    lib.fspad_verify_step.argtypes = [vp, vp, ci] + [vp] * 10 + [ci, ci] + [vp] * 6
    lib.fspad_verify_step_host.argtypes = [vp] * 12 + [ci, ci] + [vp] * 6
    lib.fspad_tree_build.argtypes = [vp] * 5 + [ci, ci, ci] + [vp] * 6
    lib.fspad_draft_expand.argtypes = [vp] * 4 + [ci] * 6 + [vp] * 6
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().fspad_strerror(code).decode()


def _ptr(t: Optional[torch.Tensor], dtype, device_type: str = "cuda"):
    if t is None:
        return None
    if t.dtype != dtype:
        raise TypeError("expected %s, got %s" % (dtype, t.dtype))
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    if t.device.type != device_type:
        raise ValueError("tensor must live on %s, not %s" % (device_type, t.device))
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


class Context:
    """Owns an `fspad_ctx` on the current CUDA device."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, vocab: int, max_len: int, max_nodes: int = 64,
                 n_layers: int = 1, max_batch: int = 1, head_dim: int = 128, softmax_scale: float = 0.0):
        if not torch.cuda.is_available():
            raise RuntimeError("fspad needs a CUDA device (there is no CPU fallback)")
        self.cfg = FspadConfig(n_q_heads, n_kv_heads, head_dim, max_nodes, vocab, n_layers, max_len,
                               max_batch, softmax_scale)
        self._h = ctypes.c_void_p()
        rc = load().fspad_create(ctypes.byref(self.cfg), ctypes.byref(self._h))
        if rc != 0:
            raise FspadError(rc, "fspad_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            load().fspad_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- raw return-code forms (used by the boundary tests) -----------------
    def status(self, stream=None) -> int:
        return load().fspad_status(self._h, _stream(stream))

    def launch_count(self) -> int:
        return int(load().fspad_launch_count(self._h))

    def check(self, stream=None):
        rc = self.status(stream)
        if rc != 0:
            raise FspadError(rc, "device status")

    def selftest_wait_timeout(self, polls: int = 64, stream=None) -> int:
        return load().fspad_selftest_wait_timeout(self._h, polls, _stream(stream))

    # -- the three operations --------------------------------------------------
    def tree_attn(self, q, k_cache, v_cache, tree_k, tree_v, parent, prefix_len, out=None, stream=None):
        B, N = q.shape[0], q.shape[1]
        if out is None:
            out = torch.empty_like(q)
        bf = torch.bfloat16
        rc = load().fspad_tree_attn(self._h, _ptr(q, bf), _ptr(k_cache, bf), _ptr(v_cache, bf),
                                    _ptr(tree_k, bf), _ptr(tree_v, bf), _ptr(parent, torch.int32),
                                    _ptr(prefix_len, torch.int32), N, B, _ptr(out, bf), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_tree_attn")
        return out

    def tree_accept(self, target_logits, draft_probs, draft_tokens, parent, temperature, uniforms,
                    accepted_path=None, n_accepted=None, bonus_token=None, stream=None):
        B, N = target_logits.shape[0], target_logits.shape[1]
        dev = target_logits.device
        if accepted_path is None:
            accepted_path = torch.empty((B, self.cfg.max_nodes), dtype=torch.int32, device=dev)
        if n_accepted is None:
            n_accepted = torch.empty((B,), dtype=torch.int32, device=dev)
        if bonus_token is None:
            bonus_token = torch.empty((B,), dtype=torch.int32, device=dev)
        f32, i32 = torch.float32, torch.int32
        rc = load().fspad_tree_accept(self._h, _ptr(target_logits, f32), _ptr(draft_probs, f32),
                                      _ptr(draft_tokens, i32), _ptr(parent, i32), _ptr(temperature, f32),
                                      _ptr(uniforms, f32), N, B, _ptr(accepted_path, i32),
                                      _ptr(n_accepted, i32), _ptr(bonus_token, i32), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_tree_accept")
        return accepted_path, n_accepted, bonus_token

    def accept_stats(self, logits, temperature, rows_per_seq, out=None, stream=None):
        rows = logits.shape[0]
        dev = logits.device
        if out is None:
            out = (torch.empty((rows,), dtype=torch.float32, device=dev),
                   torch.empty((rows,), dtype=torch.float64, device=dev),
                   torch.empty((rows,), dtype=torch.int32, device=dev))
        elif out == "scan_only":      # the streaming pass alone; partials stay in the context
            out = (None, None, None)
        row_max, row_sum, row_arg = out
        rc = load().fspad_accept_stats(self._h, _ptr(logits, torch.float32), _ptr(temperature, torch.float32),
                                       rows, rows_per_seq, _ptr(row_max, torch.float32),
                                       _ptr(row_sum, torch.float64), _ptr(row_arg, torch.int32),
                                       _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_accept_stats")
        return row_max, row_sum, row_arg

    def tree_attn_paged(self, q, k_pool, v_pool, block_table, tree_k, tree_v, parent, prefix_len, out=None, stream=None):
        """Attention over a cache kept as pools of 128-row blocks [n_blocks][Hkv][128][d] and a block table [B][blocks]."""
        B, N = q.shape[0], q.shape[1]
        if out is None:
            out = torch.empty_like(q)
        bf, i32 = torch.bfloat16, torch.int32
        rc = load().fspad_tree_attn_paged(self._h, _ptr(q, bf), _ptr(k_pool, bf), _ptr(v_pool, bf), _ptr(block_table, i32),
                                          block_table.shape[1], k_pool.shape[0], _ptr(tree_k, bf), _ptr(tree_v, bf),
                                          _ptr(parent, i32), _ptr(prefix_len, i32), N, B, _ptr(out, bf), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_tree_attn_paged")
        return out

    def kv_compact_paged(self, pool, block_table, accepted_path, n_accepted, prefix_len, new_len=None, stream=None):
        """Compaction on a pool [layers][2][n_blocks][Hkv][128][d] addressed through block_table [B][blocks]."""
        B = prefix_len.shape[0]
        i32 = torch.int32
        if new_len is None:
            new_len = torch.empty((B,), dtype=i32, device=pool.device)
        rc = load().fspad_kv_compact_paged(self._h, _ptr(pool, torch.bfloat16), _ptr(block_table, i32), block_table.shape[1],
                                           pool.shape[2], _ptr(accepted_path, i32), _ptr(n_accepted, i32), _ptr(prefix_len, i32),
                                           B, _ptr(new_len, i32), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_kv_compact_paged")
        return new_len

    def lm_head_stats(self, hidden, lm_head, temperature, rows_per_seq, logits_out=None, out=None, stream=None):
        """hidden [rows][H], lm_head [V][H] (bf16, device) -> (row_max, row_sum, row_arg); logits_out, if given,
        receives the fp32 logits [rows][V]."""
        rows, H = hidden.shape
        dev = hidden.device
        if out is None:
            out = (torch.empty((rows,), dtype=torch.float32, device=dev), torch.empty((rows,), dtype=torch.float64, device=dev),
                   torch.empty((rows,), dtype=torch.int32, device=dev))
        bf = torch.bfloat16
        rc = load().fspad_lm_head_stats(self._h, _ptr(hidden, bf), _ptr(lm_head, bf), H, rows, rows_per_seq,
                                        _ptr(temperature, torch.float32), _ptr(logits_out, torch.float32),
                                        _ptr(out[0], torch.float32), _ptr(out[1], torch.float64), _ptr(out[2], torch.int32),
                                        _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_lm_head_stats")
        return out

    def lm_head_accept(self, hidden, lm_head, draft_probs, draft_tokens, parent, temperature, uniforms, logits=None,
                       accepted_path=None, n_accepted=None, bonus_token=None, stream=None):
        """hidden [B][N][H] -> acceptance result, the logits' scan fused behind the LM-head product."""
        B, N, H = hidden.shape
        dev = hidden.device
        i32, f32, bf = torch.int32, torch.float32, torch.bfloat16
        if accepted_path is None:
            accepted_path = torch.empty((B, self.cfg.max_nodes), dtype=i32, device=dev)
        if n_accepted is None:
            n_accepted = torch.empty((B,), dtype=i32, device=dev)
        if bonus_token is None:
            bonus_token = torch.empty((B,), dtype=i32, device=dev)
        rc = load().fspad_lm_head_accept(self._h, _ptr(hidden, bf), _ptr(lm_head, bf), H, _ptr(draft_probs, f32),
                                         _ptr(draft_tokens, i32), _ptr(parent, i32), _ptr(temperature, f32),
                                         _ptr(uniforms, f32), N, B, _ptr(logits, f32), _ptr(accepted_path, i32),
                                         _ptr(n_accepted, i32), _ptr(bonus_token, i32), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_lm_head_accept")
        return accepted_path, n_accepted, bonus_token

    def feature_sampler(self, f, e, w_up, w_gate, w_down, inter=None, eta=None, workspace=None, stream=None):
        """f, e [rows][H]; w_up, w_gate [I][H]; w_down [H][I] (bf16, device) -> (eta [rows][H], inter [rows][I])."""
        rows, H = f.shape
        I = w_up.shape[0]
        bf = torch.bfloat16
        if inter is None:
            inter = torch.empty((rows, I), dtype=bf, device=f.device)
        if eta is None:
            eta = torch.empty((rows, H), dtype=bf, device=f.device)
        need = load().fspad_feature_sampler_workspace_bytes(rows, H, I)
        if workspace is None:
            workspace = torch.empty((need,), dtype=torch.uint8, device=f.device)
        rc = load().fspad_feature_sampler(self._h, _ptr(f, bf), _ptr(e, bf), _ptr(w_up, bf), _ptr(w_gate, bf), _ptr(w_down, bf),
                                          rows, H, I, _ptr(inter, bf), _ptr(eta, bf), _ptr(workspace, torch.uint8),
                                          workspace.numel(), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_feature_sampler")
        return eta, inter

    def kv_append(self, cache, tree_kv, accepted_path, n_accepted, prefix_len, new_len=None, stream=None):
        """cache [layers][2][B][Hkv][max_len][d], tree_kv [layers][2][B][Hkv][N][d]: accepted rows written behind the prefix."""
        B = prefix_len.shape[0]
        i32 = torch.int32
        if new_len is None:
            new_len = torch.empty((B,), dtype=i32, device=cache.device)
        rc = load().fspad_kv_append(self._h, _ptr(cache, torch.bfloat16), _ptr(tree_kv, torch.bfloat16), _ptr(accepted_path, i32),
                                    _ptr(n_accepted, i32), _ptr(prefix_len, i32), tree_kv.shape[4], B, _ptr(new_len, i32),
                                    _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_kv_append")
        return new_len

    def kv_compact(self, cache, accepted_path, n_accepted, prefix_len, new_len=None, stream=None):
        B = prefix_len.shape[0]
        if new_len is None:
            new_len = torch.empty((B,), dtype=torch.int32, device=cache.device)
        i32 = torch.int32
        rc = load().fspad_kv_compact(self._h, _ptr(cache, torch.bfloat16), _ptr(accepted_path, i32),
                                     _ptr(n_accepted, i32), _ptr(prefix_len, i32), B, _ptr(new_len, i32),
                                     _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_kv_compact")
        return new_len

    def tree_build(self, cand_parent, cand_token, cand_logp, root_token, n_nodes, out=None, anc=None, stream=None):
        """Candidates [B][C] (device) -> (parent, token, cand) [B][n_nodes] and n_out [B]; `anc`, if given,
        is an int64 tensor [B][n_nodes] that receives the ancestor masks (bit patterns of uint64)."""
        B, C = cand_parent.shape
        i32 = torch.int32
        if out is None:
            dev = cand_parent.device
            out = tuple(torch.empty((B, n_nodes), dtype=i32, device=dev) for _ in range(3)) + \
                (torch.empty((B,), dtype=i32, device=dev),)
        parent, token, cand, n_out = out
        rc = load().fspad_tree_build(self._h, _ptr(cand_parent, i32), _ptr(cand_token, i32),
                                     _ptr(cand_logp, torch.float32), _ptr(root_token, i32), C, n_nodes, B,
                                     _ptr(parent, i32), _ptr(token, i32), _ptr(cand, i32),
                                     _ptr(anc, torch.int64) if anc is not None else None, _ptr(n_out, i32),
                                     _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_tree_build")
        return parent, token, cand, n_out

    def draft_expand(self, logprobs, frontier_logp, frontier_cand, top_k, width, base, cand_parent, cand_token,
                     cand_logp, next_cand=None, next_logp=None, stream=None):
        """One draft step: logprobs [B][F][V] (device) -> new candidates written into cand_* [B][cap] at
        base .. base + F*top_k - 1; returns (next_cand, next_logp) [B][width]."""
        B, F, V = logprobs.shape
        assert V == self.cfg.vocab
        i32, f32 = torch.int32, torch.float32
        if next_cand is None:
            next_cand = torch.empty((B, width), dtype=i32, device=logprobs.device)
        if next_logp is None:
            next_logp = torch.empty((B, width), dtype=f32, device=logprobs.device)
        rc = load().fspad_draft_expand(self._h, _ptr(logprobs, f32), _ptr(frontier_logp, f32), _ptr(frontier_cand, i32),
                                       F, top_k, width, base, cand_parent.shape[1], B, _ptr(cand_parent, i32),
                                       _ptr(cand_token, i32), _ptr(cand_logp, f32), _ptr(next_cand, i32),
                                       _ptr(next_logp, f32), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_draft_expand")
        return next_cand, next_logp

    def verify_step(self, cache, q, tree_k, tree_v, parent, prefix_len, target_logits, draft_probs, draft_tokens,
                    temperature, uniforms, attn_out, accepted_path, n_accepted, bonus_token, new_len, attn_layer=0,
                    stream=None):
        """The whole verify step on device tensors: attention (second stream of the context) beside
        acceptance, then compaction; outputs are written in place."""
        B, N = q.shape[0], q.shape[1]
        bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
        rc = load().fspad_verify_step(
            self._h, _ptr(cache, bf), attn_layer, _ptr(q, bf), _ptr(tree_k, bf), _ptr(tree_v, bf), _ptr(parent, i32),
            _ptr(prefix_len, i32), _ptr(target_logits, f32), _ptr(draft_probs, f32), _ptr(draft_tokens, i32),
            _ptr(temperature, f32), _ptr(uniforms, f32), N, B, _ptr(attn_out, bf), _ptr(accepted_path, i32),
            _ptr(n_accepted, i32), _ptr(bonus_token, i32), _ptr(new_len, i32), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_verify_step")
        return attn_out, accepted_path, n_accepted, bonus_token, new_len

    def verify_step_host(self, cache, q, tree_k, tree_v, parent, prefix_len, target_logits, draft_probs,
                         draft_tokens, temperature, uniforms, attn_out, accepted_path, n_accepted,
                         bonus_token, new_len, stream=None):
        """All tensors except `cache` are HOST tensors (pinned recommended); outputs are written in place."""
        B, N = q.shape[0], q.shape[1]
        bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
        h = "cpu"
        rc = load().fspad_verify_step_host(
            self._h, _ptr(cache, bf), _ptr(q, bf, h), _ptr(tree_k, bf, h), _ptr(tree_v, bf, h),
            _ptr(parent, i32, h), _ptr(prefix_len, i32, h), _ptr(target_logits, f32, h),
            _ptr(draft_probs, f32, h), _ptr(draft_tokens, i32, h), _ptr(temperature, f32, h),
            _ptr(uniforms, f32, h), N, B, _ptr(attn_out, bf, h), _ptr(accepted_path, i32, h),
            _ptr(n_accepted, i32, h), _ptr(bonus_token, i32, h), _ptr(new_len, i32, h), _stream(stream))
        if rc != 0:
            raise FspadError(rc, "fspad_verify_step_host")
        return attn_out, accepted_path, n_accepted, bonus_token, new_len


def accept_stats_noalloc(logits, temperature, rows_per_seq, out, stream=None) -> int:
    """Context-free per-node scan for callers that may not allocate device memory; the
    caller supplies the three output tensors.  Returns the library's status code."""
    rows, vocab = logits.shape
    row_max, row_sum, row_arg = out
    return load().fspad_accept_stats_noalloc(_ptr(logits, torch.float32), _ptr(temperature, torch.float32), rows,
                                             rows_per_seq, vocab, _ptr(row_max, torch.float32),
                                             _ptr(row_sum, torch.float64), _ptr(row_arg, torch.int32),
                                             _stream(stream))


def bf16_tensor(bits, device="cuda"):
    """numpy uint16 bit patterns -> torch.bfloat16 tensor on `device` (no value conversion)."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device) if device != "cpu" else t


def bf16_bits(t: torch.Tensor):
    """torch.bfloat16 tensor -> numpy uint16 bit patterns."""
    import numpy as np
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
