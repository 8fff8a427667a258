"""Pins for the oracle's cache append of the accepted path: a numpy fancy-index brute force, the equivalence with
"write every tree row behind the prefix, then compact" (the pinned compaction), hand-placed rows, and what must
stay untouched."""
import numpy as np
import pytest

import oracle
from paper_2408_15562_b200 import synth


def _case(paths_list, N=8, layers=3, Hkv=2, d=4, Ls=None, slack=2):
    B = len(paths_list)
    Ls = np.asarray(Ls if Ls is not None else [3 + b for b in range(B)], np.int32)
    max_len = int(Ls.max()) + N + slack
    cache = synth.hashed_u16((layers, 2, B, Hkv, max_len, d), 7)
    tree = synth.hashed_u16((layers, 2, B, Hkv, N, d), 8)
    paths = np.full((B, N), -1, np.int32)
    n_acc = np.zeros(B, np.int32)
    for b, p in enumerate(paths_list):
        paths[b, :len(p)] = p
        n_acc[b] = len(p)
    return cache, tree, paths, n_acc, Ls


CASES = [
    [[0, 1, 2, 3]],
    [[0, 2, 5]],
    [[0, 4, 5, 6, 7]],
    [[0], [0, 3, 7], [0, 1, 6]],
]


@pytest.mark.parametrize("paths", CASES)
def test_append_matches_fancy_index(paths):
    cache, tree, p, n, L = _case(paths)
    want = cache.copy()
    for b in range(len(paths)):
        k = int(n[b])
        want[:, :, b, :, L[b]:L[b] + k, :] = tree[:, :, b][:, :, :, p[b, :k], :]
    got = cache.copy()
    new_len = oracle.kv_append(got, tree, p, n, L)
    np.testing.assert_array_equal(got, want)
    np.testing.assert_array_equal(new_len, L + n)


@pytest.mark.parametrize("paths", CASES)
def test_append_equals_scatter_then_compact_on_the_kept_rows(paths):
    """Writing all N tree rows behind the prefix and compacting leaves the same rows [0, L + n) as the append;
    beyond them the append leaves the cache as it was, the other route leaves tree rows."""
    cache, tree, p, n, L = _case(paths)
    via = cache.copy()
    N = tree.shape[4]
    for b in range(len(paths)):
        via[:, :, b, :, L[b]:L[b] + N, :] = tree[:, :, b]
    oracle.kv_compact(via, p, n, L)
    got = cache.copy()
    oracle.kv_append(got, tree, p, n, L)
    for b in range(len(paths)):
        end = int(L[b] + n[b])
        np.testing.assert_array_equal(got[:, :, b, :, :end], via[:, :, b, :, :end])
        np.testing.assert_array_equal(got[:, :, b, :, end:], cache[:, :, b, :, end:])


def test_hand_placed_rows_and_layer_kv_head_addressing():
    # every (layer, K/V, head) slice carries its own constant so that a slip in any index shows
    layers, Hkv, N, d, L = 2, 3, 5, 2, 4
    cache = np.zeros((layers, 2, 1, Hkv, L + N, d), np.uint16)
    tree = np.zeros((layers, 2, 1, Hkv, N, d), np.uint16)
    for l in range(layers):
        for kv in range(2):
            for h in range(Hkv):
                for j in range(N):
                    tree[l, kv, 0, h, j, :] = 1000 * l + 100 * kv + 10 * h + j + 1
    p = np.array([[0, 2, 4, -1, -1]], np.int32)
    oracle.kv_append(cache, tree, p, np.array([3], np.int32), np.array([L], np.int32))
    for l in range(layers):
        for kv in range(2):
            for h in range(Hkv):
                base = 1000 * l + 100 * kv + 10 * h + 1
                assert cache[l, kv, 0, h, L:, 0].tolist() == [base, base + 2, base + 4, 0, 0]
                assert not cache[l, kv, 0, h, :L].any()


def test_empty_path_writes_nothing_and_bad_inputs_are_refused():
    cache, tree, p, n, L = _case([[0, 1]])
    got = cache.copy()
    new_len = oracle.kv_append(got, tree, p, np.zeros(1, np.int32), L)
    np.testing.assert_array_equal(got, cache)
    np.testing.assert_array_equal(new_len, L)
    bad = p.copy()
    bad[0, 1] = tree.shape[4]
    with pytest.raises(RuntimeError):
        oracle.kv_append(cache.copy(), tree, bad, n, L)
    with pytest.raises(RuntimeError):
        oracle.kv_append(cache.copy(), tree, p, n, np.array([cache.shape[4] - 1], np.int32))
