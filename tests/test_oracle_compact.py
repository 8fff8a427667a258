"""Pins for the oracle's accepted-path KV compaction: a numpy brute force on a
copied cache, the identity path, overlapping moves and the worst case."""
import numpy as np
import pytest

import oracle
from paper_2408_15562_b200 import synth


def _brute(cache, paths, n_acc, L):
    old = cache.copy()
    new = cache.copy()
    for b in range(cache.shape[2]):
        for j in range(int(n_acc[b])):
            new[:, :, b, :, L[b] + j, :] = old[:, :, b, :, L[b] + paths[b, j], :]
    return new


def _case(paths_list, N=8, layers=3, Hkv=2, d=4, Ls=None):
    B = len(paths_list)
    Ls = np.asarray(Ls if Ls is not None else [3 + b for b in range(B)], np.int32)
    max_len = int(Ls.max()) + N + 2
    cache = synth.hashed_u16((layers, 2, B, Hkv, max_len, d), 42)
    paths = np.full((B, N), -1, np.int32)
    n_acc = np.zeros(B, np.int32)
    for b, p in enumerate(paths_list):
        paths[b, :len(p)] = p
        n_acc[b] = len(p)
    return cache, paths, n_acc, Ls


@pytest.mark.parametrize("paths", [
    [[0, 1, 2, 3]],                 # identity: nothing moves
    [[0, 2, 5]],                    # overlapping: row 2 is both a source and a destination
    [[0, 4, 5, 6, 7]],              # worst case: deepest path at the end of the tree
    [[0], [0, 3, 7], [0, 1, 6]],    # batch with different lengths
])
def test_compaction_matches_brute_force(paths):
    cache, p, n, L = _case(paths)
    want = _brute(cache, p, n, L)
    got = cache.copy()
    new_len = oracle.kv_compact(got, p, n, L)
    np.testing.assert_array_equal(got, want)
    np.testing.assert_array_equal(new_len, L + n)


def test_identity_path_is_a_no_op_and_outside_rows_untouched():
    cache, p, n, L = _case([[0, 1, 2]])
    got = cache.copy()
    oracle.kv_compact(got, p, n, L)
    np.testing.assert_array_equal(got, cache)
    cache, p, n, L = _case([[0, 3, 6]])
    got = cache.copy()
    oracle.kv_compact(got, p, n, L)
    Lb = int(L[0])
    np.testing.assert_array_equal(got[:, :, 0, :, :Lb], cache[:, :, 0, :, :Lb])
    np.testing.assert_array_equal(got[:, :, 0, :, Lb + 3:], cache[:, :, 0, :, Lb + 3:])
    np.testing.assert_array_equal(got[:, :, 0, :, Lb + 1], cache[:, :, 0, :, Lb + 3])
    np.testing.assert_array_equal(got[:, :, 0, :, Lb + 2], cache[:, :, 0, :, Lb + 6])


def test_random_paths_on_generated_trees():
    rng = np.random.default_rng(2)
    for _ in range(5):
        N = 20
        parents = [synth.pruned_tree(rng, N, 5, 3) for _ in range(3)]
        paths = [list(synth.random_path(rng, par)) for par in parents]
        cache, p, n, L = _case(paths, N=N, layers=2, Hkv=3, d=8, Ls=[0, 5, 9])
        want = _brute(cache, p, n, L)
        oracle.kv_compact(cache, p, n, L)
        np.testing.assert_array_equal(cache, want)
