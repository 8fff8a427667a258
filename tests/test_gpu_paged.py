"""Attention and compaction on a paged cache (`fspad_tree_attn_paged`, `fspad_kv_compact_paged`) against the
oracle: the paged cache is turned into the contiguous cache it stands for (oracle.paged_to_contiguous) and the
oracle's contiguous functions give the expected result.  Attention within the stated bound, compaction bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth
from tests import helpers

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


def _paged_from(inp, rng, spare=3):
    """Pools [n_blocks][Hkv][128][d] for K and V holding inp's cache in scrambled blocks, and the table."""
    B, Hkv, max_len, d = inp.k_cache.shape
    nb = (max_len + 127) // 128
    pad = nb * 128 - max_len
    kc = np.concatenate([inp.k_cache, synth.hashed_u16((B, Hkv, pad, d), 5)], axis=2) if pad else inp.k_cache
    vc = np.concatenate([inp.v_cache, synth.hashed_u16((B, Hkv, pad, d), 6)], axis=2) if pad else inp.v_cache
    n_blocks = B * nb + spare
    table = rng.permutation(n_blocks)[:B * nb].reshape(B, nb).astype(np.int32)
    k_pool = synth.hashed_u16((n_blocks, Hkv, 128, d), 7) & 0x3FFF          # filler: finite values
    v_pool = synth.hashed_u16((n_blocks, Hkv, 128, d), 8) & 0x3FFF
    oracle.contiguous_to_paged(kc, table, k_pool)
    oracle.contiguous_to_paged(vc, table, v_pool)
    return k_pool, v_pool, table


def _check_attn(inp, seed, aliased, seqs=None):
    rng = np.random.default_rng(seed)
    k_pool, v_pool, table = _paged_from(inp, rng)
    B, N = inp.parent.shape
    ctx = helpers.make_ctx(inp)
    b16 = binding.bf16_tensor
    out = ctx.tree_attn_paged(b16(inp.q), b16(k_pool), b16(v_pool), helpers.dev(table), None if aliased else b16(inp.tree_k),
                              None if aliased else b16(inp.tree_v), helpers.dev(inp.parent), helpers.dev(inp.prefix_len))
    ctx.check()
    kc = oracle.paged_to_contiguous(k_pool, table)
    vc = oracle.paged_to_contiguous(v_pool, table)
    for b in (range(B) if seqs is None else seqs):
        sl = slice(b, b + 1)
        ref = oracle.tree_attn(inp.q[sl], np.ascontiguousarray(kc[sl]), np.ascontiguousarray(vc[sl]),
                               None if aliased else inp.tree_k[sl], None if aliased else inp.tree_v[sl], inp.parent[sl],
                               inp.prefix_len[sl])
        mx, mean = helpers.attn_errors(out[sl], ref)
        assert mx <= 1e-2 and mean <= 1e-3, (b, mx, mean)


@pytest.mark.parametrize("aliased", [False, True])
@pytest.mark.parametrize("prefix", [(0, 0), (100, 130), (128, 128), (250, 700)])
def test_attention_small_shapes(prefix, aliased):
    w = synth.scaled(W["llama3_8b_2k"], batch=3, n_q_heads=8, n_kv_heads=2, prefix=prefix, n_nodes=19, depth=4, branch=3,
                     vocab=16, temperatures=(0.0, 0.0, 0.0))
    inp = synth.generate(w, 2, with_accept=False)
    if prefix[1] < 64:
        for arr in (inp.v_cache, inp.tree_v):      # few keys: outputs as large as single draws; keep them of order one
            nz = arr & 0x7FFF != 0
            arr[nz] -= np.uint16(2 << 7)
    _check_attn(inp, 1, aliased)


def test_attention_headline_and_ragged_batch():
    _check_attn(synth.generate(W["llama3_8b_2k"], 0, with_accept=False), 3, False)
    inp = synth.generate(W["batch16_ragged"], 0, with_accept=False)
    _check_attn(inp, 4, True, seqs=[0, int(np.argmin(inp.prefix_len)), int(np.argmax(inp.prefix_len))])


def test_compaction_paged():
    rng = np.random.default_rng(9)
    B, N, Hkv, nl, nb = 4, 60, 3, 3, 5
    parents = [synth.pruned_tree(rng, N, 6, 10) for _ in range(B)]
    paths = np.full((B, 64), -1, np.int32)
    n = np.zeros(B, np.int32)
    for b, par in enumerate(parents):
        p = synth.random_path(rng, par)
        paths[b, :len(p)] = p
        n[b] = len(p)
    paths[0, :9] = np.arange(9) * 2              # a long overlapping path that crosses a block boundary
    n[0] = 9
    L = np.array([120, 0, 300, 517], np.int32)   # sequence 0: tree rows straddle blocks 0 and 1
    n_blocks = B * nb + 2
    table = rng.permutation(n_blocks)[:B * nb].reshape(B, nb).astype(np.int32)
    pool = synth.hashed_u16((nl, 2, n_blocks, Hkv, 128, 128), 3)
    ctx = binding.Context(6, Hkv, 16, nb * 128, max_nodes=64, n_layers=nl, max_batch=B)
    dpool = binding.bf16_tensor(pool)
    new_len = ctx.kv_compact_paged(dpool, helpers.dev(table), helpers.dev(paths), helpers.dev(n), helpers.dev(L))
    ctx.check()
    cache = oracle.paged_to_contiguous(pool, table)
    want_len = oracle.kv_compact(cache, paths, n, L)
    want_pool = pool.copy()
    oracle.contiguous_to_paged(cache, table, want_pool)
    np.testing.assert_array_equal(binding.bf16_bits(dpool), want_pool)
    np.testing.assert_array_equal(new_len.cpu().numpy(), want_len)


def test_bad_table_entry_is_reported_and_stays_in_bounds():
    w = synth.scaled(W["llama3_8b_2k"], batch=1, n_q_heads=8, n_kv_heads=2, prefix=(200, 200), n_nodes=10, depth=3, branch=3,
                     vocab=16)
    inp = synth.generate(w, 0, with_accept=False)
    k_pool, v_pool, table = _paged_from(inp, np.random.default_rng(0))
    table[0, 1] = k_pool.shape[0] + 5
    ctx = helpers.make_ctx(inp)
    b16 = binding.bf16_tensor
    ctx.tree_attn_paged(b16(inp.q), b16(k_pool), b16(v_pool), helpers.dev(table), b16(inp.tree_k), b16(inp.tree_v),
                        helpers.dev(inp.parent), helpers.dev(inp.prefix_len))
    assert ctx.status() == -5
    pool = binding.bf16_tensor(synth.hashed_u16((1, 2, k_pool.shape[0], 2, 128, 128), 1))
    paths = np.full((1, 10), -1, np.int32)
    paths[0, :3] = [0, 2, 5]
    ctx2 = binding.Context(8, 2, 16, table.shape[1] * 128, max_nodes=10, n_layers=1, max_batch=1)
    ctx2.kv_compact_paged(pool, helpers.dev(table), helpers.dev(paths), helpers.dev(np.array([3], np.int32)),
                          helpers.dev(np.array([126], np.int32)))       # rows 126.. reach the bad block
    assert ctx2.status() == -5
