"""CUDA KV compaction (through the C ABI) against the oracle: bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth
from tests import helpers

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


def _run_case(cache, paths, n_acc, L, Hq, max_nodes):
    n_layers, _, B, Hkv, max_len, d = cache.shape
    ctx = binding.Context(Hq, Hkv, 16, max_len, max_nodes=max_nodes, n_layers=n_layers, max_batch=B)
    dc = binding.bf16_tensor(cache)
    new_len = ctx.kv_compact(dc, helpers.dev(paths), helpers.dev(n_acc), helpers.dev(L))
    ctx.check()
    want = cache.copy()
    want_len = oracle.kv_compact(want, paths, n_acc, L)
    np.testing.assert_array_equal(binding.bf16_bits(dc), want)
    np.testing.assert_array_equal(new_len.cpu().numpy(), want_len)


def _paths(rng, parents, max_nodes):
    B = len(parents)
    paths = np.full((B, max_nodes), -1, np.int32)
    n = np.zeros(B, np.int32)
    for b, par in enumerate(parents):
        p = synth.random_path(rng, par)
        paths[b, :len(p)] = p
        n[b] = len(p)
    return paths, n


@pytest.mark.parametrize("case", ["identity", "overlap", "worst", "root_only"])
def test_hand_paths(case):
    N = 12
    p = {"identity": [0, 1, 2, 3], "overlap": [0, 2, 5], "worst": [0, 7, 8, 9, 10, 11], "root_only": [0]}[case]
    cache = synth.hashed_u16((3, 2, 1, 2, 40, 128), 7)
    paths = np.full((1, N), -1, np.int32)
    paths[0, :len(p)] = p
    _run_case(cache, paths, np.array([len(p)], np.int32), np.array([9], np.int32), 4, N)


def test_random_paths_batched_multi_layer():
    rng = np.random.default_rng(5)
    for it in range(4):
        B, N = 5, 60
        parents = [synth.pruned_tree(rng, N, 6, 10) for _ in range(B)]
        paths, n = _paths(rng, parents, 64)
        L = rng.integers(0, 100, B).astype(np.int32)
        cache = synth.hashed_u16((4, 2, B, 3, 100 + 64, 128), it)
        _run_case(cache, paths, n, L, 6, 64)


def test_long_chain_path_uses_several_row_batches():
    N = 64
    cache = synth.hashed_u16((2, 2, 2, 2, 200, 128), 3)
    paths = np.full((2, N), -1, np.int32)
    paths[0, :30] = np.arange(30) * 2            # every second node: 30 overlapping moves
    paths[0, 0] = 0
    paths[1, :64] = np.arange(64)                # identity over the whole tree
    _run_case(cache, paths, np.array([30, 64], np.int32), np.array([17, 100], np.int32), 2, N)


@pytest.mark.parametrize("n", [3, 5, 7, 9, 15, 17, 31])
def test_odd_lengths_where_one_half_warp_reads_what_the_other_writes(n):
    """Paths [0, 2, 4, ...] and [0, 1, 3, 5, ...] of odd length: in every batch of eight moves the
    destination row of one half-warp is the source row of the other."""
    N = 64
    cache = synth.hashed_u16((2, 2, 2, 3, 150, 128), n)
    paths = np.full((2, N), -1, np.int32)
    paths[0, :n] = np.arange(n) * 2
    paths[1, :n] = np.concatenate([[0], np.arange(1, n) * 2 - 1])
    _run_case(cache, paths, np.array([n, n], np.int32), np.array([11, 70], np.int32), 3, N)


def test_full_size_batch16_32_layers_sampled_slices():
    """Configuration of the batched ragged workload: 32 layers x 16 sequences x 8 kv
    heads, max_len 4160.  The device cache is filled by a hash of the flat index;
    sampled (layer, K/V, sequence, head) slices are compared bit-exactly with the
    oracle's result on the same slice, and the untouched regions are checked whole."""
    w = W["batch16_ragged"]
    inp = synth.generate(w, 0, with_attention=False, with_accept=False)
    rng = np.random.default_rng(9)
    B, Hkv, max_len, nl = w.batch, w.n_kv_heads, inp.max_len, w.n_layers
    paths, n = _paths(rng, list(inp.parent), 64)
    L = inp.prefix_len
    ctx = binding.Context(w.n_q_heads, Hkv, 16, max_len, max_nodes=64, n_layers=nl, max_batch=B)
    per_layer = 2 * B * Hkv * max_len * 128
    bits = torch.empty(nl * per_layer, dtype=torch.int16, device="cuda")
    for l in range(nl):
        idx = torch.arange(l * per_layer, (l + 1) * per_layer, dtype=torch.int64, device="cuda")
        bits[l * per_layer:(l + 1) * per_layer] = ((idx * 2654435761 + (idx >> 13) * 40503) & 0x7FFF).to(torch.int16)
        del idx
    cache = bits.view(torch.bfloat16).view(nl, 2, B, Hkv, max_len, 128)
    before = cache.clone()
    new_len = ctx.kv_compact(cache, helpers.dev(paths), helpers.dev(n), helpers.dev(L))
    ctx.check()
    np.testing.assert_array_equal(new_len.cpu().numpy(), L + n)
    for _ in range(24):
        l, kv, b, h = int(rng.integers(nl)), int(rng.integers(2)), int(rng.integers(B)), int(rng.integers(Hkv))
        sl = binding.bf16_bits(before[l, kv, b, h])[None, None, None, None].copy()
        sl = np.broadcast_to(sl, (1, 2, 1, 1, max_len, 128)).copy()
        oracle.kv_compact(sl, paths[b:b + 1], n[b:b + 1], L[b:b + 1])
        np.testing.assert_array_equal(binding.bf16_bits(cache[l, kv, b, h]), sl[0, 0, 0, 0])
    # prefix rows and rows after the tree are untouched everywhere
    for b in range(B):
        assert torch.equal(cache[:, :, b, :, :int(L[b])].view(torch.int16), before[:, :, b, :, :int(L[b])].view(torch.int16))
        assert torch.equal(cache[:, :, b, :, int(L[b]) + 64:].view(torch.int16), before[:, :, b, :, int(L[b]) + 64:].view(torch.int16))


def test_invalid_path_is_reported_and_stays_in_bounds():
    cache = synth.hashed_u16((1, 2, 1, 2, 40, 128), 1)
    ctx = binding.Context(4, 2, 16, 40, max_nodes=12, n_layers=1, max_batch=1)
    dc = binding.bf16_tensor(cache)
    paths = np.full((1, 12), -1, np.int32)
    paths[0, :3] = [0, 5, 3]                      # not increasing
    ctx.kv_compact(dc, helpers.dev(paths), helpers.dev(np.array([3], np.int32)), helpers.dev(np.array([4], np.int32)))
    assert ctx.status() == -5
