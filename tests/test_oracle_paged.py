"""Pins for the paged-cache helpers of the oracle: a paged cache means the contiguous cache obtained by reading
every sequence's blocks in table order (checked against numpy's fancy indexing and by hand), and writing a
contiguous cache back into its blocks inverts that."""
import numpy as np

import oracle


def test_gather_matches_numpy_indexing_and_hand_case():
    rng = np.random.default_rng(0)
    pool = rng.integers(0, 65536, size=(2, 2, 7, 3, 128, 8), dtype=np.uint16)     # [layers][2][n_blocks][Hkv][128][d]
    table = np.array([[4, 0, 6], [2, 5, 1]], np.int32)
    got = oracle.paged_to_contiguous(pool, table)
    assert got.shape == (2, 2, 2, 3, 384, 8)
    want = np.moveaxis(pool[:, :, table], [2, 3, 4, 5], [2, 4, 3, 5]).reshape(2, 2, 2, 3, 384, 8)   # [.., B, blocks, Hkv, 128, d] -> [.., B, Hkv, blocks*128, d]
    np.testing.assert_array_equal(got, want)
    # by hand: row 130 of sequence 1 is row 2 of block 5
    np.testing.assert_array_equal(got[1, 0, 1, 2, 130], pool[1, 0, 5, 2, 2])
    np.testing.assert_array_equal(got[0, 1, 0, 0, 383], pool[0, 1, 6, 0, 127])


def test_scatter_inverts_gather():
    rng = np.random.default_rng(1)
    pool = rng.integers(0, 65536, size=(3, 2, 9, 2, 128, 4), dtype=np.uint16)
    table = np.array([[8, 3], [0, 7], [5, 1]], np.int32)
    cache = oracle.paged_to_contiguous(pool, table)
    cache[..., 17, :] ^= 0xFFFF
    pool2 = pool.copy()
    oracle.contiguous_to_paged(cache, table, pool2)
    np.testing.assert_array_equal(oracle.paged_to_contiguous(pool2, table), cache)
    untouched = [b for b in range(9) if b not in table.ravel()]
    np.testing.assert_array_equal(pool2[:, :, untouched], pool[:, :, untouched])
