"""ctypes front end of the fp64 CPU oracle (`fspad_oracle.c`).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg use it; the CUDA library and its Python binding never
import this package, and this package imports nothing of theirs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fspad_oracle.c")
_LIB = os.path.join(_HERE, "libfspad_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, OpenMP over independent units)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp,
                               _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a: Optional[np.ndarray], dtype):
    if a is None:
        return None
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def set_threads(n: int) -> None:
    """Number of OpenMP threads the oracle's parallel loops use from now on (timing only: the
    loops run over independent units, results do not depend on it)."""
    os.environ["OMP_NUM_THREADS"] = str(n)
    lib()                                             # the OpenMP runtime is in the process once the oracle is
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
    except OSError:
        pass


def tree_attn(q, k_cache, v_cache, tree_k, tree_v, parent, prefix_len, scale: Optional[float] = None):
    """fp64 tree-masked attention; bf16 inputs as uint16 bit arrays. Returns [B][N][Hq][d] float64."""
    B, N, Hq, d = q.shape
    _, Hkv, max_len, _ = k_cache.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = np.empty((B, N, Hq, d), dtype=np.float64)
    rc = lib().oracle_tree_attn(_p(q, np.uint16), _p(k_cache, np.uint16), _p(v_cache, np.uint16),
                                _p(tree_k, np.uint16), _p(tree_v, np.uint16), _p(parent, np.int32),
                                _p(prefix_len, np.int32), B, N, Hq, Hkv, d, max_len,
                                ctypes.c_double(scale), _p(out, np.float64))
    if rc != 0:
        raise RuntimeError("oracle_tree_attn failed: %d" % rc)
    return out


def row_stats(logits: np.ndarray, T: float = 1.0):
    R, V = logits.shape
    m = np.empty(R, np.float64)
    s = np.empty(R, np.float64)
    a = np.empty(R, np.int32)
    lib().oracle_row_stats(_p(logits, np.float32), R, V, ctypes.c_double(T), _p(m, np.float64),
                           _p(s, np.float64), _p(a, np.int32))
    return m, s, a


def lm_head_stats(hidden, weight, T: float = 1.0, want_logits: bool = False):
    """fp64 LM head (hidden [R][H] x weight [V][H]^T, bf16 bit patterns) followed by the row statistics of
    its logits.  Returns a dict: max, sum, arg, gap (maximum minus runner-up) [R] and, on request, logits [R][V]."""
    R, H = hidden.shape
    V, H2 = weight.shape
    assert H == H2
    m = np.empty(R, np.float64)
    s = np.empty(R, np.float64)
    a = np.empty(R, np.int32)
    gap = np.empty(R, np.float64)
    z = np.empty((R, V), np.float64) if want_logits else None
    rc = lib().oracle_lm_head_stats(_p(hidden, np.uint16), _p(weight, np.uint16), R, H, V, ctypes.c_double(T),
                                    _p(z, np.float64), _p(m, np.float64), _p(s, np.float64), _p(a, np.int32),
                                    _p(gap, np.float64))
    if rc != 0:
        raise RuntimeError("oracle_lm_head_stats failed: %d" % rc)
    return {"max": m, "sum": s, "arg": a, "gap": gap, "logits": z}


def feature_sampler(f, e, wup, wgate, wdown, want_inter: bool = False):
    """fp64 Feature Sampler forward: eta = Wdown (silu(Wgate e) * (Wup f)) + f.  f, e [R][H]; wup, wgate [I][H];
    wdown [H][I] (bf16 bit patterns).  Returns eta [R][H] float64 (and the intermediate [R][I] on request)."""
    R, H = f.shape
    I = wup.shape[0]
    assert e.shape == (R, H) and wup.shape == (I, H) and wgate.shape == (I, H) and wdown.shape == (H, I)
    eta = np.empty((R, H), np.float64)
    inter = np.empty((R, I), np.float64) if want_inter else None
    rc = lib().oracle_feature_sampler(_p(f, np.uint16), _p(e, np.uint16), _p(wup, np.uint16), _p(wgate, np.uint16),
                                      _p(wdown, np.uint16), R, H, I, _p(eta, np.float64), _p(inter, np.float64))
    if rc != 0:
        raise RuntimeError("oracle_feature_sampler failed: %d" % rc)
    return (eta, inter) if want_inter else eta


def tree_accept(target_logits, draft_probs, draft_tokens, parent, temperature, uniforms,
                force: Optional[np.ndarray] = None):
    """Lossless tree acceptance. Returns a dict with accepted_path [B][N] (-1 padded),
    n_accepted [B], bonus_token [B] and the fp64 decision trace."""
    B, N, V = target_logits.shape
    path = np.empty((B, N), np.int32)
    n_acc = np.empty(B, np.int32)
    bonus = np.empty(B, np.int32)
    trq = np.empty((B, N), np.float64)
    tp = np.empty((B, N), np.float64)
    binfo = np.empty((B, 6), np.float64)
    rc = lib().oracle_tree_accept(_p(target_logits, np.float32), _p(draft_probs, np.float32),
                                  _p(draft_tokens, np.int32), _p(parent, np.int32),
                                  _p(temperature, np.float32), _p(uniforms, np.float32),
                                  _p(force, np.int32), B, N, V, _p(path, np.int32),
                                  _p(n_acc, np.int32), _p(bonus, np.int32), _p(trq, np.float64),
                                  _p(tp, np.float64), _p(binfo, np.float64))
    if rc != 0:
        raise RuntimeError("oracle_tree_accept failed: %d" % rc)
    return {"accepted_path": path, "n_accepted": n_acc, "bonus_token": bonus,
            "trace_rq": trq, "trace_p": tp, "bonus_info": binfo}


def kv_compact(cache: np.ndarray, accepted_path, n_accepted, prefix_len):
    """In-place accepted-path compaction of cache [layers][2][B][Hkv][max_len][d] (uint16)."""
    n_layers, two, B, Hkv, max_len, d = cache.shape
    assert two == 2
    new_len = np.empty(B, np.int32)
    rc = lib().oracle_kv_compact(_p(cache, np.uint16), _p(accepted_path, np.int32),
                                 _p(n_accepted, np.int32), _p(prefix_len, np.int32), n_layers, B,
                                 Hkv, max_len, d, accepted_path.shape[1], _p(new_len, np.int32))
    if rc != 0:
        raise RuntimeError("oracle_kv_compact failed: %d" % rc)
    return new_len


def kv_append(cache: np.ndarray, tree_kv: np.ndarray, accepted_path, n_accepted, prefix_len):
    """In place: the accepted path's rows of tree_kv [layers][2][B][Hkv][N][d] written behind the prefix of
    cache [layers][2][B][Hkv][max_len][d] (both uint16); returns new_len."""
    n_layers, two, B, Hkv, max_len, d = cache.shape
    assert two == 2 and tree_kv.shape[:4] == cache.shape[:4] and tree_kv.shape[5] == d
    N = tree_kv.shape[4]
    new_len = np.empty(B, np.int32)
    rc = lib().oracle_kv_append(_p(cache, np.uint16), _p(tree_kv, np.uint16), _p(accepted_path, np.int32),
                                _p(n_accepted, np.int32), _p(prefix_len, np.int32), n_layers, B, Hkv, max_len,
                                N, d, accepted_path.shape[1], _p(new_len, np.int32))
    if rc != 0:
        raise RuntimeError("oracle_kv_append failed: %d" % rc)
    return new_len


def paged_to_contiguous(pool: np.ndarray, table: np.ndarray) -> np.ndarray:
    """What a paged cache means: pool [..., n_blocks, Hkv, 128, d] and table [B][blocks] -> the contiguous cache
    [..., B, Hkv, blocks * 128, d] in which row r of sequence b is row r % 128 of block table[b][r // 128]."""
    B, nb = table.shape
    lead = pool.shape[:-4]
    _, Hkv, bs, d = pool.shape[-4:]
    out = np.empty(lead + (B, Hkv, nb * bs, d), dtype=pool.dtype)
    for b in range(B):
        for i in range(nb):
            out[..., b, :, i * bs:(i + 1) * bs, :] = pool[..., int(table[b, i]), :, :, :]
    return out


def contiguous_to_paged(cache: np.ndarray, table: np.ndarray, pool: np.ndarray) -> None:
    """The inverse: writes the rows of the contiguous cache [..., B, Hkv, blocks * 128, d] into their blocks of pool."""
    B, nb = table.shape
    bs = pool.shape[-2]
    for b in range(B):
        for i in range(nb):
            pool[..., int(table[b, i]), :, :, :] = cache[..., b, :, i * bs:(i + 1) * bs, :]


def tree_build(cand_parent, cand_token, cand_logp, root_token, n_nodes: int):
    """Final stage of the dynamic token tree: keep the n_nodes - 1 most probable candidates and
    flatten them breadth-first behind the root.  Arrays [B][C]; returns parent, token, cand [B][N]
    and n_out [B]; `valid` is False when the joint probabilities were not monotone along a path."""
    cand_parent = np.ascontiguousarray(cand_parent, np.int32)
    B, C = cand_parent.shape
    parent = np.empty((B, n_nodes), np.int32)
    token = np.empty((B, n_nodes), np.int32)
    cand = np.empty((B, n_nodes), np.int32)
    n_out = np.empty(B, np.int32)
    anc = np.empty((B, n_nodes), np.uint64)
    rc = lib().oracle_tree_build(_p(cand_parent, np.int32), _p(cand_token, np.int32), _p(cand_logp, np.float32),
                                 _p(root_token, np.int32), B, C, n_nodes, _p(parent, np.int32),
                                 _p(token, np.int32), _p(cand, np.int32), _p(anc, np.uint64), _p(n_out, np.int32))
    if rc not in (0, -3):
        raise RuntimeError("oracle_tree_build failed: %d" % rc)
    return {"parent": parent, "token": token, "cand": cand, "anc": anc, "n_out": n_out, "valid": rc == 0}


def draft_expand(logprobs, frontier_logp, frontier_cand, top_k: int, width: int, base: int,
                 cand_parent, cand_token, cand_logp):
    """One draft step of the dynamic tree: per-row top-k, joint log-probabilities, next frontier.
    logprobs [B][F][V]; the candidate arrays [B][cap] are updated in place at base .. base + F*top_k - 1.
    Returns (next_cand [B][width], next_logp [B][width])."""
    logprobs = np.ascontiguousarray(logprobs, np.float32)
    B, F, V = logprobs.shape
    cap = cand_parent.shape[1]
    next_cand = np.empty((B, width), np.int32)
    next_logp = np.empty((B, width), np.float32)
    rc = lib().oracle_draft_expand(_p(logprobs, np.float32), _p(np.ascontiguousarray(frontier_logp, np.float32), np.float32),
                                   _p(np.ascontiguousarray(frontier_cand, np.int32), np.int32), B, F, V, top_k, width,
                                   base, cap, _p(cand_parent, np.int32), _p(cand_token, np.int32),
                                   _p(cand_logp, np.float32), _p(next_cand, np.int32), _p(next_logp, np.float32))
    if rc != 0:
        raise RuntimeError("oracle_draft_expand failed: %d" % rc)
    return next_cand, next_logp
