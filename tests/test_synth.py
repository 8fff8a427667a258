"""Host-side checks of the synthetic workload generator (shapes, tree validity)."""
import numpy as np

from paper_2408_15562_b200 import synth


def _valid_tree(parent):
    assert parent[0] == -1
    assert all(0 <= parent[i] < i for i in range(1, len(parent)))


def test_bfs_tree_tiny_config_levels():
    par = synth.bfs_tree(26, 3)
    _valid_tree(par)
    assert synth.tree_depth(par) == 4            # levels 1 + 3 + 9 + 13


def test_pruned_tree_has_requested_size_and_depth():
    for seed in range(20):
        par = synth.pruned_tree(np.random.default_rng(seed), 60, 6, 10)
        _valid_tree(par)
        assert len(par) == 60 and synth.tree_depth(par) == 6
        # breadth-first numbering: parents are non-decreasing
        assert all(par[i] <= par[i + 1] for i in range(1, 59))


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, 1.00390625, 1.005859375, -2.5, 3.14159], np.float32)
    b = synth.f32_to_bf16_bits(x)
    y = synth.bf16_bits_to_f32(b)
    assert y[0] == 1.0 and y[3] == -2.5
    assert y[1] == 1.0                            # halfway case rounds to even mantissa
    assert y[2] == np.float32(1.0078125)
    assert abs(y[4] - 3.14159) < 2 ** -7


def test_generate_small_workload_shapes_and_determinism():
    w = synth.scaled(synth.WORKLOADS["llama3_8b_2k"], prefix=(40, 40), vocab=500, n_nodes=20, depth=4,
                     branch=3)
    a = synth.generate(w)
    b = synth.generate(w)
    assert a.q.shape == (1, 20, 32, 128) and a.k_cache.shape == (1, 8, 40 + 64, 128)
    assert a.target_logits.shape == (1, 20, 500) and a.draft_probs.shape == (1, 20, 500)
    np.testing.assert_array_equal(a.q, b.q)
    np.testing.assert_array_equal(a.draft_tokens, b.draft_tokens)
    np.testing.assert_allclose(a.draft_probs.sum(-1), 1.0, atol=1e-5)
    ch = synth.children_lists(a.parent[0])
    for i, c in enumerate(ch):                    # sibling tokens are distinct (drawn without replacement)
        toks = a.draft_tokens[0, c]
        assert len(set(toks.tolist())) == len(c)
    assert (a.uniforms >= 0).all() and (a.uniforms < 1).all()
    cache = synth.make_cache(a, 2)
    np.testing.assert_array_equal(cache[0, 0, 0, :, 40:60], a.tree_k[0])
