"""CUDA cache append of the accepted path (through the C ABI) against the oracle: bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth
from tests import helpers

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


def _run_case(cache, tree, paths, n_acc, L, Hq, max_nodes):
    n_layers, _, B, Hkv, max_len, d = cache.shape
    ctx = binding.Context(Hq, Hkv, 16, max_len, max_nodes=max_nodes, n_layers=n_layers, max_batch=B)
    dc, dt = binding.bf16_tensor(cache), binding.bf16_tensor(tree)
    new_len = ctx.kv_append(dc, dt, helpers.dev(paths), helpers.dev(n_acc), helpers.dev(L))
    ctx.check()
    want = cache.copy()
    want_len = oracle.kv_append(want, tree, paths, n_acc, L)
    np.testing.assert_array_equal(binding.bf16_bits(dc), want)
    np.testing.assert_array_equal(binding.bf16_bits(dt), tree)
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


@pytest.mark.parametrize("case", ["identity", "gaps", "worst", "root_only", "empty"])
def test_hand_paths(case):
    N = 12
    p = {"identity": [0, 1, 2, 3], "gaps": [0, 2, 5], "worst": [0, 7, 8, 9, 10, 11], "root_only": [0], "empty": []}[case]
    cache = synth.hashed_u16((3, 2, 1, 2, 40, 128), 7)
    tree = synth.hashed_u16((3, 2, 1, 2, N, 128), 8)
    paths = np.full((1, N), -1, np.int32)
    paths[0, :len(p)] = p
    _run_case(cache, tree, paths, np.array([len(p)], np.int32), np.array([9], np.int32), 4, N)


def test_random_paths_batched_multi_layer():
    rng = np.random.default_rng(5)
    for it in range(4):
        B, N = 5, 60
        parents = [synth.pruned_tree(rng, N, 6, 10) for _ in range(B)]
        paths, n = _paths(rng, parents, 64)
        L = rng.integers(0, 100, B).astype(np.int32)
        cache = synth.hashed_u16((4, 2, B, 3, 100 + 64, 128), it)
        tree = synth.hashed_u16((4, 2, B, 3, N, 128), 100 + it)
        _run_case(cache, tree, paths, n, L, 6, 64)


@pytest.mark.parametrize("n", [1, 7, 8, 9, 16, 17, 64, 200])
def test_path_lengths_around_the_row_batches_and_wide_trees(n):
    """Eight rows are in flight per warp: lengths at and around multiples of eight, up to a 200-node chain of a
    256-node tree; the cache ends exactly at L + n for the second sequence."""
    N = 256 if n > 64 else 64
    max_len = max(50 + n, N)
    L = np.array([3, max_len - n], np.int32)
    cache = synth.hashed_u16((2, 2, 2, 2, max_len, 128), n)
    tree = synth.hashed_u16((2, 2, 2, 2, N, 128), 1000 + n)
    paths = np.full((2, N), -1, np.int32)
    paths[0, :n] = np.arange(n)
    paths[1, :n] = np.concatenate([[0], np.arange(N - n + 1, N)])[:n]
    _run_case(cache, tree, paths, np.array([n, n], np.int32), L, 2, N)


def test_full_size_batch16_32_layers_sampled_slices():
    """The batched ragged workload: 32 layers x 16 sequences x 8 kv heads, max_len 4160, 60-node trees.  Sampled
    (layer, K/V, sequence, head) slices are compared with the oracle on the same slice; everything outside
    rows [L, L + n) is checked whole against the cache as it was."""
    w = W["batch16_ragged"]
    inp = synth.generate(w, 0, with_attention=False, with_accept=False)
    rng = np.random.default_rng(9)
    B, Hkv, max_len, nl, N = w.batch, w.n_kv_heads, inp.max_len, w.n_layers, w.n_nodes
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
    tidx = torch.arange(nl * 2 * B * Hkv * N * 128, dtype=torch.int64, device="cuda")
    tree = ((tidx * 40503 + (tidx >> 11) * 2654435761 + 12345) & 0x7FFF).to(torch.int16).view(torch.bfloat16).view(nl, 2, B, Hkv, N, 128)
    del tidx
    before = cache.clone()
    new_len = ctx.kv_append(cache, tree, helpers.dev(paths), helpers.dev(n), helpers.dev(L))
    ctx.check()
    np.testing.assert_array_equal(new_len.cpu().numpy(), L + n)
    for _ in range(24):
        l, kv, b, h = int(rng.integers(nl)), int(rng.integers(2)), int(rng.integers(B)), int(rng.integers(Hkv))
        sl = binding.bf16_bits(before[l, kv, b, h])[None, None, None, None].copy()
        sl = np.broadcast_to(sl, (1, 2, 1, 1, max_len, 128)).copy()
        tr = binding.bf16_bits(tree[l, kv, b, h])[None, None, None, None].copy()
        tr = np.broadcast_to(tr, (1, 2, 1, 1, N, 128)).copy()
        oracle.kv_append(sl, tr, paths[b:b + 1], n[b:b + 1], L[b:b + 1])
        np.testing.assert_array_equal(binding.bf16_bits(cache[l, kv, b, h]), sl[0, 0, 0, 0])
    for b in range(B):
        lo, hi = int(L[b]), int(L[b] + n[b])
        assert torch.equal(cache[:, :, b, :, :lo].view(torch.int16), before[:, :, b, :, :lo].view(torch.int16))
        assert torch.equal(cache[:, :, b, :, hi:].view(torch.int16), before[:, :, b, :, hi:].view(torch.int16))


def test_invalid_inputs_are_reported_and_stay_in_bounds():
    cache = synth.hashed_u16((1, 2, 1, 2, 40, 128), 1)
    tree = synth.hashed_u16((1, 2, 1, 2, 12, 128), 2)
    ctx = binding.Context(4, 2, 16, 40, max_nodes=12, n_layers=1, max_batch=1)
    dc, dt = binding.bf16_tensor(cache), binding.bf16_tensor(tree)
    paths = np.full((1, 12), -1, np.int32)
    paths[0, :3] = [0, 12, 3]                     # node 12 does not exist
    ctx.kv_append(dc, dt, helpers.dev(paths), helpers.dev(np.array([3], np.int32)), helpers.dev(np.array([4], np.int32)))
    assert ctx.status() == -5
    paths[0, :3] = [0, 1, 2]
    ctx.kv_append(dc, dt, helpers.dev(paths), helpers.dev(np.array([3], np.int32)), helpers.dev(np.array([38], np.int32)))
    assert ctx.status() == -5                     # L + n > max_len
    np.testing.assert_array_equal(binding.bf16_bits(dc)[:, :, :, :, 38:], cache[:, :, :, :, 38:])
