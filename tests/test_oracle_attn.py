"""Pins for the oracle's tree-masked attention.

Each check compares the oracle with something that is not the oracle: a dense
causal attention written here in numpy, a per-path brute force that turns every
node into an ordinary sequence, and closed-form special cases.
"""
import numpy as np
import pytest

import oracle
from paper_2408_15562_b200 import synth


def _rand_case(rng, B, N, Hq, Hkv, d, Lmax, parent, with_tree_arrays=True):
    L = rng.integers(0, Lmax + 1, size=B).astype(np.int32)
    max_len = Lmax + N + 3
    q = synth.normal_bf16(rng, (B, N, Hq, d))
    kc = synth.normal_bf16(rng, (B, Hkv, max_len, d))
    vc = synth.normal_bf16(rng, (B, Hkv, max_len, d))
    tk = synth.normal_bf16(rng, (B, Hkv, N, d))
    tv = synth.normal_bf16(rng, (B, Hkv, N, d))
    par = np.tile(parent, (B, 1)).astype(np.int32)
    return q, kc, vc, tk, tv, par, L


def _dense_last_row_attention(qrow, K, Vv, scale):
    """Plain softmax attention of one query over all rows of K/V (float64)."""
    s = (K @ qrow) * scale
    s = s - s.max()
    p = np.exp(s)
    return (p[:, None] * Vv).sum(0) / p.sum()


def _f(x):
    return synth.bf16_bits_to_f32(x).astype(np.float64)


def _path(parent, i):
    out = []
    while i >= 0:
        out.append(i)
        i = int(parent[i])
    return out[::-1]


@pytest.mark.parametrize("tree", ["pruned", "bfs", "star"])
def test_per_path_brute_force(tree):
    """Every node == last position of a plain sequence prefix ++ root-path."""
    rng = np.random.default_rng(11)
    B, N, Hq, Hkv, d = 2, 13, 4, 2, 16
    parent = {"pruned": synth.pruned_tree(rng, N, 4, 3), "bfs": synth.bfs_tree(N, 3),
              "star": synth.star_tree(N)}[tree]
    q, kc, vc, tk, tv, par, L = _rand_case(rng, B, N, Hq, Hkv, d, 9, parent)
    scale = 0.37
    out = oracle.tree_attn(q, kc, vc, tk, tv, par, L, scale)
    G = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            g = h // G
            for i in range(N):
                pth = _path(parent, i)
                K = np.concatenate([_f(kc[b, g, :L[b]]), _f(tk[b, g, pth])])
                Vv = np.concatenate([_f(vc[b, g, :L[b]]), _f(tv[b, g, pth])])
                ref = _dense_last_row_attention(_f(q[b, i, h]), K, Vv, scale)
                np.testing.assert_allclose(out[b, i, h], ref, rtol=0, atol=1e-12)


def test_chain_tree_is_causal_attention():
    """parent[i] = i-1: the N tree queries are the last N rows of dense causal attention."""
    rng = np.random.default_rng(5)
    B, N, Hq, Hkv, d, Lmax = 1, 7, 2, 1, 8, 6
    parent = synth.chain_tree(N)
    q, kc, vc, tk, tv, par, L = _rand_case(rng, B, N, Hq, Hkv, d, Lmax, parent)
    L[:] = Lmax
    out = oracle.tree_attn(q, kc, vc, tk, tv, par, L)
    scale = 1.0 / np.sqrt(d)
    T = Lmax + N
    for h in range(Hq):
        K = np.concatenate([_f(kc[0, 0, :Lmax]), _f(tk[0, 0])])
        Vv = np.concatenate([_f(vc[0, 0, :Lmax]), _f(tv[0, 0])])
        Q = np.zeros((T, d))
        Q[Lmax:] = _f(q[0, :, h])
        S = (Q @ K.T) * scale
        S[np.triu_indices(T, 1)] = -np.inf           # causal mask
        S -= S.max(1, keepdims=True)
        P = np.exp(S)
        P /= P.sum(1, keepdims=True)
        O = P @ Vv
        np.testing.assert_allclose(out[0, :, h], O[Lmax:], rtol=0, atol=1e-12)


def test_tree_rows_read_from_cache_when_no_tree_arrays():
    rng = np.random.default_rng(6)
    B, N, Hq, Hkv, d = 2, 6, 2, 2, 8
    parent = synth.bfs_tree(N, 2)
    q, kc, vc, tk, tv, par, L = _rand_case(rng, B, N, Hq, Hkv, d, 5, parent)
    for b in range(B):
        kc[b, :, L[b]:L[b] + N] = tk[b]
        vc[b, :, L[b]:L[b] + N] = tv[b]
    a = oracle.tree_attn(q, kc, vc, tk, tv, par, L)
    c = oracle.tree_attn(q, kc, vc, None, None, par, L)
    np.testing.assert_array_equal(a, c)


def test_equal_values_give_that_value_and_single_key():
    """All V rows equal -> output is that row (weights sum to 1); N=1, L=0 -> the root's own V row."""
    rng = np.random.default_rng(7)
    B, N, Hq, Hkv, d = 1, 5, 2, 1, 8
    parent = synth.bfs_tree(N, 2)
    q, kc, vc, tk, tv, par, L = _rand_case(rng, B, N, Hq, Hkv, d, 4, parent)
    vc[:] = vc[0, 0, 0]
    tv[:] = vc[0, 0, 0]
    out = oracle.tree_attn(q, kc, vc, tk, tv, par, L)
    np.testing.assert_allclose(out, np.broadcast_to(_f(vc[0, 0, 0]), out.shape), atol=1e-14)

    q1, kc1, vc1, tk1, tv1, par1, L1 = _rand_case(rng, 1, 1, 2, 1, 8, 0, synth.chain_tree(1))
    out1 = oracle.tree_attn(q1, kc1, vc1, tk1, tv1, par1, L1)
    np.testing.assert_array_equal(out1[0, 0, 0], _f(tv1[0, 0, 0]))
    np.testing.assert_array_equal(out1[0, 0, 1], _f(tv1[0, 0, 0]))


def test_sibling_relabelling_permutes_outputs():
    """Swapping the indices of two sibling leaves only swaps their output rows."""
    rng = np.random.default_rng(8)
    N, Hq, Hkv, d = 6, 2, 1, 8
    parent = np.array([-1, 0, 0, 1, 1, 2], dtype=np.int32)
    q, kc, vc, tk, tv, par, L = _rand_case(rng, 1, N, Hq, Hkv, d, 4, parent)
    a = oracle.tree_attn(q, kc, vc, tk, tv, par, L)
    perm = np.array([0, 1, 2, 4, 3, 5])          # nodes 3 and 4 are sibling leaves
    b = oracle.tree_attn(np.ascontiguousarray(q[:, perm]), kc, vc, np.ascontiguousarray(tk[:, :, perm]),
                         np.ascontiguousarray(tv[:, :, perm]), par, L)
    np.testing.assert_allclose(b, a[:, perm], atol=1e-14)


def test_gqa_head_mapping_is_contiguous_groups():
    """With G=2, query heads 0,1 use kv head 0 and heads 2,3 use kv head 1."""
    rng = np.random.default_rng(9)
    N, d = 4, 8
    parent = synth.chain_tree(N)
    q, kc, vc, tk, tv, par, L = _rand_case(rng, 1, N, 4, 2, d, 3, parent)
    q[:, :, 1] = q[:, :, 0]
    q[:, :, 3] = q[:, :, 0]
    q[:, :, 2] = q[:, :, 0]
    out = oracle.tree_attn(q, kc, vc, tk, tv, par, L)
    np.testing.assert_array_equal(out[:, :, 0], out[:, :, 1])
    np.testing.assert_array_equal(out[:, :, 2], out[:, :, 3])
    assert np.abs(out[:, :, 0] - out[:, :, 2]).max() > 1e-3
