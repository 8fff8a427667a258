"""The oracle on trees of more than 64 nodes (the verify step accepts up to 256): the same independent
checks as for small trees - every node as a plain sequence (dense softmax in numpy), greedy acceptance against
the naive marking of fully matching root paths, compaction against a copy - at sizes where a 64-bit mask word
no longer holds a tree."""
import numpy as np
import pytest

import oracle
from paper_2408_15562_b200 import synth
from tests.test_oracle_attn import _dense_last_row_attention, _f, _path, _rand_case
from tests.test_oracle_accept import _naive_greedy


@pytest.mark.parametrize("tree,N", [("pruned", 130), ("bfs", 200), ("chain", 70)])
def test_attention_per_path_brute_force(tree, N):
    rng = np.random.default_rng(21)
    B, Hq, Hkv, d = 1, 2, 1, 16
    parent = {"pruned": lambda: synth.pruned_tree(rng, N, 7, 10), "bfs": lambda: synth.bfs_tree(N, 3),
              "chain": lambda: synth.chain_tree(N)}[tree]()
    q, kc, vc, tk, tv, par, L = _rand_case(rng, B, N, Hq, Hkv, d, 5, parent)
    out = oracle.tree_attn(q, kc, vc, tk, tv, par, L, 0.29)
    for h in range(Hq):
        for i in range(0, N, 3):
            pth = _path(parent, i)
            K = np.concatenate([_f(kc[0, 0, :L[0]]), _f(tk[0, 0, pth])])
            Vv = np.concatenate([_f(vc[0, 0, :L[0]]), _f(tv[0, 0, pth])])
            want = _dense_last_row_attention(_f(q[0, i, h]), K, Vv, 0.29)
            np.testing.assert_allclose(out[0, i, h], want, rtol=1e-11, atol=1e-12)


def test_greedy_equals_naive_marking_on_a_wide_tree():
    rng = np.random.default_rng(5)
    N, V = 180, 40
    for _ in range(4):
        parent = synth.pruned_tree(rng, N, 7, 10)
        logits = rng.standard_normal((1, N, V)).astype(np.float32)
        tokens = np.zeros((1, N), np.int32)
        for i, ch in enumerate(synth.children_lists(parent)):       # children carry the best tokens of their parent's row, shuffled
            if ch:
                top = np.argsort(-logits[0, i], kind="stable")[:len(ch)]
                tokens[0, ch] = rng.permutation(top)
        r = oracle.tree_accept(logits, None, tokens, parent[None].astype(np.int32), np.zeros(1, np.float32), None)
        want_path, want_bonus = _naive_greedy(logits[0], tokens[0], parent)
        k = int(r["n_accepted"][0])
        assert list(r["accepted_path"][0, :k]) == want_path and int(r["bonus_token"][0]) == want_bonus
        assert k >= 2                                                # the best token is among the children: the walk moves


def test_compaction_of_a_long_path():
    rng = np.random.default_rng(2)
    cache = synth.hashed_u16((2, 2, 1, 2, 400, 8), 4)
    N = 256
    path = np.full((1, N), -1, np.int32)
    sel = np.sort(rng.choice(np.arange(1, N), size=99, replace=False))
    path[0, 0] = 0
    path[0, 1:100] = sel
    want = cache.copy()
    L = 77
    for j in range(100):
        want[:, :, 0, :, L + j] = cache[:, :, 0, :, L + path[0, j]]
    new_len = oracle.kv_compact(cache, path, np.array([100], np.int32), np.array([L], np.int32))
    np.testing.assert_array_equal(cache, want)
    assert int(new_len[0]) == L + 100
