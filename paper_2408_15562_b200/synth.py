"""Seeded synthetic workloads for the tree-verification step.

This module only *produces inputs*: random tensors, draft trees, a stand-in
draft distribution and the random numbers the acceptance pass consumes. It
holds none of the verification arithmetic (no attention, no acceptance rule,
no compaction) and is the one module that both the CPU oracle's tests and the
CUDA path's tests/benchmark import. All arrays are host numpy arrays; bf16
tensors are carried as uint16 bit patterns (round-to-nearest-even from fp32).

The five named workloads are shaped like the paper's evaluation models
(Vicuna 7B/33B, LLaMA3-Instruct 8B/70B; 60 candidate tokens per tree, Section
"Experiments"); the draft tree is a stand-in for the dynamic-tree method the
paper adopts (Section "Preliminaries": per-step top-k, joint probability,
global top-k over all candidates).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence

import numpy as np

SEED_BASE = 24081556200
HEAD_DIM = 128


# --------------------------------------------------------------------------
# bf16 bit helpers (storage format only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rnd = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rnd) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    cfg: int                      # index used in the seed
    batch: int
    n_q_heads: int
    n_kv_heads: int
    prefix: Sequence[int]         # (lo, hi) inclusive range, or (L, L)
    n_nodes: int
    depth: int                    # tree levels including the root
    branch: int                   # children per expanded node
    tree: str                     # "bfs" (every node expanded in order) or "pruned"
    vocab: int
    logit_sigma: float
    temperatures: Sequence[float]  # one per sequence (0 = greedy)
    n_layers: int = 1
    head_dim: int = HEAD_DIM
    tail: int = 64                # spare cache rows after the longest prefix

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


WORKLOADS: Dict[str, Workload] = {
    "tiny_greedy": Workload("tiny_greedy", 1, 1, 32, 32, (256, 256), 26, 4, 3, "bfs",
                            32000, 2.0, (0.0,)),
    "llama3_8b_2k": Workload("llama3_8b_2k", 2, 1, 32, 8, (2048, 2048), 60, 6, 10, "pruned",
                             128256, 3.0, (1.0,)),
    "vicuna_33b_4k_greedy": Workload("vicuna_33b_4k_greedy", 3, 1, 52, 52, (4096, 4096), 60, 6, 10,
                                     "pruned", 32000, 3.0, (0.0,)),
    "vicuna_33b_4k_sample": Workload("vicuna_33b_4k_sample", 3, 1, 52, 52, (4096, 4096), 60, 6, 10,
                                     "pruned", 32000, 3.0, (1.0,)),
    "llama3_70b_8k": Workload("llama3_70b_8k", 4, 1, 64, 8, (8192, 8192), 60, 6, 10, "pruned",
                              128256, 3.0, (1.0,)),
    "batch16_ragged": Workload("batch16_ragged", 5, 16, 32, 8, (512, 4096), 60, 6, 10, "pruned",
                               128256, 3.0, (0.0,) * 8 + (1.0,) * 8, n_layers=32),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some sizes overridden (parity-test sizes)."""
    return replace(w, **kw)


# --------------------------------------------------------------------------
# draft trees
# --------------------------------------------------------------------------
def bfs_tree(n_nodes: int, branch: int) -> np.ndarray:
    """Every node, in index order, gets `branch` children until n_nodes exist."""
    parent = np.full(n_nodes, -1, dtype=np.int32)
    nxt, cur = 1, 0
    while nxt < n_nodes:
        for _ in range(branch):
            if nxt >= n_nodes:
                break
            parent[nxt] = cur
            nxt += 1
        cur += 1
    return parent


def chain_tree(n_nodes: int) -> np.ndarray:
    return np.arange(-1, n_nodes - 1, dtype=np.int32)


def star_tree(n_nodes: int) -> np.ndarray:
    p = np.zeros(n_nodes, dtype=np.int32)
    p[0] = -1
    return p


def pruned_tree(rng: np.random.Generator, n_nodes: int, depth: int, branch: int) -> np.ndarray:
    """Stand-in for a dynamic draft tree: expand, score, keep the best.

    Level 1 holds `branch` children of the root; every later level picks
    `branch` nodes of the previous level and gives each `branch` children.
    A candidate's score is the product of U(0,1) draws along its path (so a
    top-score cut is closed under ancestors); one root-to-deepest chain is
    forced in so the tree has exactly `depth` levels; root + the best
    n_nodes-1 candidates are kept and renumbered breadth-first.
    """
    par: List[int] = [-1]
    lvl: List[int] = [0]
    score: List[float] = [np.inf]
    prev = [0]
    for level in range(1, depth):
        if level == 1:
            expand = prev
        else:
            k = min(branch, len(prev))
            expand = [prev[i] for i in sorted(rng.choice(len(prev), size=k, replace=False))]
        new = []
        for p in expand:
            for _ in range(branch):
                par.append(p)
                lvl.append(level)
                score.append(score[p] * rng.random() if p != 0 else rng.random())
                new.append(len(par) - 1)
        prev = new
    score_arr = np.asarray(score)
    if depth > 1:
        leaf = prev[int(rng.integers(len(prev)))]
        while leaf != 0:
            score_arr[leaf] = np.inf
            leaf = par[leaf]
    n_cand = len(par)
    n_keep = min(n_nodes, n_cand)
    order = np.argsort(-score_arr, kind="stable")[:n_keep]
    keep = np.zeros(n_cand, dtype=bool)
    keep[order] = True
    # breadth-first renumbering; children of a node in descending score
    children: Dict[int, List[int]] = {}
    for c in range(1, n_cand):
        if keep[c]:
            assert keep[par[c]]
            children.setdefault(par[c], []).append(c)
    new_id = {0: 0}
    out_parent = [-1]
    queue = [0]
    while queue:
        u = queue.pop(0)
        for c in sorted(children.get(u, []), key=lambda c: -score_arr[c]):
            new_id[c] = len(out_parent)
            out_parent.append(new_id[u])
            queue.append(c)
    return np.asarray(out_parent, dtype=np.int32)


def children_lists(parent: np.ndarray) -> List[List[int]]:
    ch: List[List[int]] = [[] for _ in range(len(parent))]
    for i in range(1, len(parent)):
        ch[int(parent[i])].append(i)
    return ch


def tree_depth(parent: np.ndarray) -> int:
    d = np.zeros(len(parent), dtype=np.int64)
    for i in range(1, len(parent)):
        d[i] = d[parent[i]] + 1
    return int(d.max()) + 1


# --------------------------------------------------------------------------
# the stand-in draft model: a noisy copy of the target distribution
# --------------------------------------------------------------------------
def _draft_distribution(rng: np.random.Generator, logits_row: np.ndarray) -> np.ndarray:
    z = logits_row.astype(np.float64) + rng.standard_normal(logits_row.shape[0])
    z -= z.max()
    e = np.exp(z)
    return (e / e.sum()).astype(np.float32)


def _draw_without_replacement(rng: np.random.Generator, probs: np.ndarray, m: int) -> np.ndarray:
    """m tokens drawn one after another from probs, each removed once drawn."""
    w = probs.astype(np.float64).copy()
    out = np.empty(m, dtype=np.int32)
    for t in range(m):
        c = np.cumsum(w)
        x = int(np.searchsorted(c, rng.random() * c[-1], side="right"))
        x = min(x, len(w) - 1)
        while w[x] == 0.0:       # landed on an exhausted token through rounding
            x = int(np.argmax(w))
        out[t] = x
        w[x] = 0.0
    return out


# --------------------------------------------------------------------------
# full input sets
# --------------------------------------------------------------------------
@dataclass
class VerifyInputs:
    workload: Workload
    seed: int
    max_len: int
    prefix_len: np.ndarray        # [B] int32
    parent: np.ndarray            # [B][N] int32
    q: np.ndarray                 # [B][N][Hq][d] bf16 bits
    k_cache: np.ndarray           # [B][Hkv][max_len][d] bf16 bits (layer 0; tree rows at L..L+N-1)
    v_cache: np.ndarray
    tree_k: np.ndarray            # [B][Hkv][N][d] bf16 bits
    tree_v: np.ndarray
    target_logits: np.ndarray     # [B][N][V] fp32
    draft_probs: Optional[np.ndarray]   # [B][N][V] fp32, None when every sequence is greedy
    draft_tokens: np.ndarray      # [B][N] int32
    temperature: np.ndarray       # [B] fp32
    uniforms: np.ndarray          # [B][N+1] fp32 in [0,1)
    extra: dict = field(default_factory=dict)


def make_tree(w: Workload, rng: np.random.Generator) -> np.ndarray:
    if w.tree == "bfs":
        return bfs_tree(w.n_nodes, w.branch)
    if w.tree == "pruned":
        return pruned_tree(rng, w.n_nodes, w.depth, w.branch)
    if w.tree == "chain":
        return chain_tree(w.n_nodes)
    if w.tree == "star":
        return star_tree(w.n_nodes)
    raise ValueError(w.tree)


def generate(w: Workload, variant: int = 0, *, with_attention: bool = True,
             with_accept: bool = True) -> VerifyInputs:
    """All inputs of one verify step for workload `w` (seeded by cfg and variant)."""
    seed = SEED_BASE + 10 * w.cfg + variant
    # independent streams, so that each part is the same whether or not the others are generated
    rng = np.random.default_rng([seed, 0])          # prefix lengths and trees
    rng_attn = np.random.default_rng([seed, 1])     # Q, K, V
    rng_acc = np.random.default_rng([seed, 2])      # logits, draft model, uniforms
    B, N, V, d = w.batch, w.n_nodes, w.vocab, w.head_dim
    lo, hi = w.prefix
    prefix_len = rng.integers(lo, hi + 1, size=B).astype(np.int32) if hi > lo \
        else np.full(B, lo, dtype=np.int32)
    max_len = int(hi) + max(w.tail, N)
    parent = np.stack([make_tree(w, rng) for _ in range(B)]).astype(np.int32)
    N = parent.shape[1]

    if with_attention:
        q = normal_bf16(rng_attn, (B, N, w.n_q_heads, d))
        k_cache = np.zeros((B, w.n_kv_heads, max_len, d), dtype=np.uint16)
        v_cache = np.zeros_like(k_cache)
        tree_k = normal_bf16(rng_attn, (B, w.n_kv_heads, N, d))
        tree_v = normal_bf16(rng_attn, (B, w.n_kv_heads, N, d))
        for b in range(B):
            L = int(prefix_len[b])
            k_cache[b, :, :L] = normal_bf16(rng_attn, (w.n_kv_heads, L, d))
            v_cache[b, :, :L] = normal_bf16(rng_attn, (w.n_kv_heads, L, d))
            k_cache[b, :, L:L + N] = tree_k[b]
            v_cache[b, :, L:L + N] = tree_v[b]
    else:
        q = k_cache = v_cache = tree_k = tree_v = np.zeros((0,), dtype=np.uint16)

    temperature = np.asarray(w.temperatures, dtype=np.float32)
    assert temperature.shape[0] == B
    any_sampling = bool((temperature > 0).any())
    if with_accept:
        logits = (rng_acc.standard_normal((B, N, V), dtype=np.float32) * np.float32(w.logit_sigma))
        draft_probs = np.zeros((B, N, V), dtype=np.float32) if any_sampling else None
        draft_tokens = np.zeros((B, N), dtype=np.int32)
        for b in range(B):
            ch = children_lists(parent[b])
            draft_tokens[b, 0] = int(rng_acc.integers(V))
            for i in range(N):
                m = len(ch[i])
                if temperature[b] > 0:
                    draft_probs[b, i] = _draft_distribution(rng_acc, logits[b, i])
                    if m:
                        draft_tokens[b, ch[i]] = _draw_without_replacement(rng_acc, draft_probs[b, i], m)
                elif m:
                    noisy = logits[b, i].astype(np.float64) + rng_acc.standard_normal(V)
                    top = np.argpartition(-noisy, min(m, V - 1))[:m]
                    top = top[np.argsort(-noisy[top], kind="stable")]
                    draft_tokens[b, ch[i]] = top.astype(np.int32)
        uniforms = rng_acc.random((B, N + 1), dtype=np.float32)
        uniforms = np.minimum(uniforms, np.float32(1.0 - 2.0 ** -24))
    else:
        logits = np.zeros((0,), dtype=np.float32)
        draft_probs = None
        draft_tokens = np.zeros((B, N), dtype=np.int32)
        uniforms = np.zeros((B, N + 1), dtype=np.float32)

    return VerifyInputs(w, seed, max_len, prefix_len, parent, q, k_cache, v_cache, tree_k, tree_v,
                        logits, draft_probs, draft_tokens, temperature, uniforms)


def hashed_u16(shape, salt: int) -> np.ndarray:
    """Deterministic 16-bit filler (an integer hash of the flat index); used for
    the cache layers that only the byte-copy compaction touches."""
    n = int(np.prod(shape))
    i = np.arange(n, dtype=np.uint64) + np.uint64((int(salt) * 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF)
    i ^= i >> np.uint64(33)
    i *= np.uint64(0xFF51AFD7ED558CCD)
    i ^= i >> np.uint64(29)
    return (i & np.uint64(0xFFFF)).astype(np.uint16).reshape(shape)


def make_cache(inp: VerifyInputs, n_layers: Optional[int] = None) -> np.ndarray:
    """Full cache [layers][2][B][Hkv][max_len][d]: layer 0 is the attention
    layer's K/V (prefix + tree rows), deeper layers carry hashed filler."""
    w = inp.workload
    n_layers = w.n_layers if n_layers is None else n_layers
    shape = (n_layers, 2) + inp.k_cache.shape
    cache = np.empty(shape, dtype=np.uint16)
    cache[0, 0] = inp.k_cache
    cache[0, 1] = inp.v_cache
    for l in range(1, n_layers):
        cache[l] = hashed_u16(shape[1:], inp.seed % 1000003 + l)
    return cache


def random_path(rng: np.random.Generator, parent: np.ndarray) -> np.ndarray:
    """A random root-to-node path (for compaction tests that skip acceptance)."""
    ch = children_lists(parent)
    path = [0]
    while ch[path[-1]] and rng.random() < 0.8:
        c = ch[path[-1]]
        path.append(int(c[int(rng.integers(len(c)))]))
    return np.asarray(path, dtype=np.int32)


# --------------------------------------------------------------------------
# candidate lists for the tree builder
# --------------------------------------------------------------------------
def tree_candidates(seed: int, batch: int, levels: int = 5, width: int = 10, branch: int = 10,
                    vocab: int = 32000, step: float = 0.0):
    """Candidate tokens as a top-k draft phase leaves them behind, listed level by level.

    Level 1: `branch` children of the root.  Every later level: `width` candidates of the previous
    level (drawn at random, not by score - choosing them is the builder's business) get `branch`
    children each.  A candidate's joint log-probability is its parent's plus log U(0,1), so it
    never grows along a path; with `step` > 0 the values are rounded down to multiples of `step`,
    which produces many ties, including children equal to their parent.  With the paper's sizes
    (levels 5, width 10, branch 10) a sequence has 10 + 4 * 100 = 410 candidates; a level never
    expands more parents than the previous level has.
    Returns cand_parent, cand_token [B][C] int32, cand_logp [B][C] float32, root_token [B] int32.
    """
    rng = np.random.default_rng([SEED_BASE % (2 ** 32), 7, seed])
    sizes = [branch]                            # candidates per level
    for _ in range(levels - 1):
        sizes.append(min(width, sizes[-1]) * branch)
    C = sum(sizes)
    cand_parent = np.empty((batch, C), np.int32)
    cand_token = rng.integers(0, vocab, size=(batch, C), dtype=np.int32)
    cand_logp = np.empty((batch, C), np.float32)
    for b in range(batch):
        lo, hi = 0, branch                      # index range of the previous level
        cand_parent[b, :branch] = -1
        cand_logp[b, :branch] = np.log(rng.random(branch))
        at = branch
        for _ in range(levels - 1):
            parents = rng.choice(np.arange(lo, hi), size=min(width, hi - lo), replace=False)
            parents.sort()
            for p in parents:
                cand_parent[b, at:at + branch] = p
                cand_logp[b, at:at + branch] = cand_logp[b, p] + np.log(rng.random(branch))
                at += branch
            lo, hi = hi, at
        assert at == C
    if step > 0:
        cand_logp = (np.floor(cand_logp / step) * step).astype(np.float32)
        for b in range(batch):                  # flooring keeps order; make sure of it in fp32
            for c in range(C):
                p = cand_parent[b, c]
                if p >= 0 and cand_logp[b, c] > cand_logp[b, p]:
                    cand_logp[b, c] = cand_logp[b, p]
    root_token = rng.integers(0, vocab, size=batch, dtype=np.int32)
    return cand_parent, cand_token, cand_logp.astype(np.float32), root_token


def draft_logprob_rows(seed: int, batch: int, n_frontier: int, vocab: int, sigma: float = 3.0, step: float = 0.0):
    """Stand-in output of one draft step: log-probabilities [B][F][V] float32 (log-softmax of
    N(0, sigma^2) logits, taken in float64).  With `step` > 0 the values are rounded down to multiples
    of `step`, which puts many equal values into every row (ties between tokens)."""
    rng = np.random.default_rng([SEED_BASE % (2 ** 32), 8, seed])
    z = rng.standard_normal((batch, n_frontier, vocab)) * sigma
    z -= z.max(-1, keepdims=True)
    lp = z - np.log(np.exp(z).sum(-1, keepdims=True))
    if step > 0:
        lp = np.floor(lp / step) * step
    return lp.astype(np.float32)


# --------------------------------------------------------------------------
# LM-head inputs (final hidden states of the tree nodes, vocabulary matrix)
# --------------------------------------------------------------------------
def lm_head_inputs(seed: int, rows: int, hidden: int, vocab: int, sigma_logit: float = 3.0):
    """Stand-in for the target's final hidden states [rows][hidden] and LM-head matrix [vocab][hidden],
    both bf16 bit patterns: hidden ~ N(0, 1), weights ~ N(0, sigma_logit^2 / hidden), so that the logits
    hidden . weight^T are ~ N(0, sigma_logit^2) like the logits of the verify workloads."""
    rng = np.random.default_rng(24081556200 + 7919 * seed + 13)
    h = normal_bf16(rng, (rows, hidden))
    w = f32_to_bf16_bits((rng.standard_normal((vocab, hidden), dtype=np.float32) *
                          np.float32(sigma_logit / np.sqrt(hidden))))
    return h, w


def feature_sampler_inputs(seed: int, rows: int, hidden: int, inter: int):
    """Stand-in inputs of the Feature Sampler (bf16 bit patterns): features f and token embeddings e [rows][hidden]
    ~ N(0, 1); Up and Gate projectors [inter][hidden] ~ N(0, 1/hidden); Down projector [hidden][inter] ~ N(0, 1/inter),
    so that every projection keeps values of order one."""
    rng = np.random.default_rng(24081556200 + 104729 * seed + 29)
    f = normal_bf16(rng, (rows, hidden))
    e = normal_bf16(rng, (rows, hidden))
    sc = np.float32(1.0 / np.sqrt(hidden))
    wup = f32_to_bf16_bits(rng.standard_normal((inter, hidden), dtype=np.float32) * sc)
    wgate = f32_to_bf16_bits(rng.standard_normal((inter, hidden), dtype=np.float32) * sc)
    wdown = f32_to_bf16_bits(rng.standard_normal((hidden, inter), dtype=np.float32) * np.float32(1.0 / np.sqrt(inter)))
    return f, e, wup, wgate, wdown

