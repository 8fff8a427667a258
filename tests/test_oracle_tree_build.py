"""Pins of the tree-builder oracle (`oracle.tree_build`): hand-worked cases, the definition of a
top-k by a library sort, brute force over all ancestor-closed subsets on tiny inputs, and the
structural invariants of a flattened tree.  CPU only."""
import itertools
import json
import os

import numpy as np
import pytest

import oracle
from paper_2408_15562_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "tree_build_hand_cases.json")


def _one(cp, ct, lp, root, n):
    r = oracle.tree_build(np.asarray([cp], np.int32), np.asarray([ct], np.int32), np.asarray([lp], np.float32),
                          np.asarray([root], np.int32), n)
    return {k: (v[0] if isinstance(v, np.ndarray) else v) for k, v in r.items()}


def test_hand_worked_cases():
    for case in json.load(open(GOLDEN))["cases"]:
        r = _one(case["cand_parent"], case["cand_token"], np.log(np.asarray(case["cand_prob"], np.float64)),
                 case["root_token"], case["n_nodes"])
        assert r["valid"], case["name"]
        assert r["n_out"] == case["n_out"], case["name"]
        for key in ("parent", "token", "cand"):
            assert r[key].tolist() == case[key], (case["name"], key, r[key].tolist())
        if "anc" in case:
            assert [int(v) for v in r["anc"]] == case["anc"], (case["name"], "anc")


@pytest.mark.parametrize("step", [0.0, 0.5])
def test_kept_set_is_the_stable_top_k(step):
    """Library definition: the first N - 1 entries of a stable descending sort."""
    for seed in range(6):
        cp, ct, lp, rt = synth.tree_candidates(seed, 3, levels=4, width=4, branch=5, vocab=100, step=step)
        for n in (2, 17, 60, 64):
            r = oracle.tree_build(cp, ct, lp, rt, n)
            assert r["valid"]
            for b in range(cp.shape[0]):
                want = set(np.argsort(-lp[b].astype(np.float64), kind="stable")[:n - 1].tolist())
                got = set(r["cand"][b, 1:r["n_out"][b]].tolist())
                assert got == want, (seed, n, b)


def test_brute_force_best_closed_subset_on_tiny_inputs():
    """Among all ancestor-closed subsets of the budgeted size, the kept one carries the most
    probability mass (values never grow along a path, so the plain top-k is such a subset)."""
    for seed in range(8):
        cp, ct, lp, rt = synth.tree_candidates(100 + seed, 1, levels=3, width=2, branch=2, vocab=50)
        cp, lp = cp[0], lp[0].astype(np.float64)
        C = len(cp)
        for n in (2, 4, 6):
            m = min(n - 1, C)
            best = -1.0
            for sub in itertools.combinations(range(C), m):
                s = set(sub)
                if all(cp[c] < 0 or cp[c] in s for c in sub):
                    best = max(best, float(np.exp(lp[list(sub)]).sum()))
            r = oracle.tree_build(cp[None], ct, lp[None].astype(np.float32), rt, n)
            kept = r["cand"][0, 1:r["n_out"][0]]
            assert abs(float(np.exp(lp[kept]).sum()) - best) <= 1e-12 * max(1.0, best), (seed, n)


def test_flattened_tree_invariants_and_path_preservation():
    for seed, step in itertools.product(range(5), (0.0, 0.25)):
        cp, ct, lp, rt = synth.tree_candidates(200 + seed, 4, step=step)
        r = oracle.tree_build(cp, ct, lp, rt, 60)
        assert r["valid"]
        for b in range(4):
            n = r["n_out"][b]
            par, tok, cand = r["parent"][b], r["token"][b], r["cand"][b]
            assert n == 60 and par[0] == -1 and tok[0] == rt[b] and cand[0] == -1
            assert all(0 <= par[i] < i for i in range(1, n))            # topological
            depth = [0] * n
            for i in range(1, n):
                depth[i] = depth[par[i]] + 1
                assert tok[i] == ct[b, cand[i]]
                # the node's parent is the node of the candidate's parent (the root for level 1)
                assert (par[i] == 0 and cp[b, cand[i]] == -1) or cand[par[i]] == cp[b, cand[i]]
            # mask: exactly the nodes on the path to the root (brute force by walking up)
            for i in range(n):
                path, j = set(), i
                while j >= 0:
                    path.add(j)
                    j = par[j]
                assert int(r["anc"][b, i]) == sum(1 << int(j) for j in path)
            keys = [(depth[i], cand[i]) for i in range(1, n)]
            assert keys == sorted(keys)                                # breadth-first, index order inside a level
            dropped = np.setdiff1d(np.arange(cp.shape[1]), cand[1:n])
            assert lp[b, dropped].max() <= lp[b, cand[1:n]].min()


def test_chain_of_candidates_gives_a_chain():
    C = 9
    cp = np.arange(-1, C - 1, dtype=np.int32)
    lp = -np.arange(1, C + 1, dtype=np.float32)
    r = _one(cp, np.arange(C), lp, 42, 6)
    assert r["parent"].tolist() == [-1, 0, 1, 2, 3, 4] and r["cand"].tolist() == [-1, 0, 1, 2, 3, 4]


def test_growing_probability_along_a_path_is_reported():
    r = _one([-1, 0, -1], [1, 2, 3], np.log([0.1, 0.5, 0.3]), 0, 3)   # child more probable than its parent
    assert not r["valid"]


# ---------------------------------------------------------------------------
# one draft step: per-row top-k, joint log-probability, next frontier
# ---------------------------------------------------------------------------
def _expand(lp, flp, fc, k, width, base, cap):
    B = lp.shape[0]
    cp = np.full((B, cap), -7, np.int32)
    ct = np.full((B, cap), -7, np.int32)
    cl = np.full((B, cap), np.nan, np.float32)
    nc, nl = oracle.draft_expand(lp, flp, fc, k, width, base, cp, ct, cl)
    return cp, ct, cl, nc, nl


def test_expand_hand_worked_cases():
    for case in json.load(open(GOLDEN))["expand_cases"]:
        lp = np.log(np.asarray([case["row_prob"]], np.float64)).astype(np.float32)
        flp = np.log(np.asarray([case["frontier_prob"]], np.float64)).astype(np.float32)
        k, base = case["top_k"], case["base"]
        n_new = len(case["frontier_cand"]) * k
        cp, ct, cl, nc, nl = _expand(lp, flp, np.asarray([case["frontier_cand"]], np.int32), k, case["width"], base,
                                     base + n_new + 2)
        assert cp[0, base:base + n_new].tolist() == case["cand_parent"], case["name"]
        assert ct[0, base:base + n_new].tolist() == case["cand_token"], case["name"]
        assert np.allclose(np.exp(cl[0, base:base + n_new].astype(np.float64)), case["cand_prob"], rtol=1e-6)
        assert nc[0].tolist() == case["next_cand"], case["name"]
        assert (cp[0, :base] == -7).all() and (cp[0, base + n_new:] == -7).all()      # nothing else written


@pytest.mark.parametrize("step", [0.0, 0.5])
def test_expand_equals_library_sorts_and_one_float_addition(step):
    for seed in range(4):
        B, F, V, k, width, base = 3, 5, 777, 7, 6, 11
        lp = synth.draft_logprob_rows(seed, B, F, V, step=step)
        rng = np.random.default_rng(seed)
        flp = (-rng.random((B, F)) * 5).astype(np.float32)
        fc = rng.integers(-1, base, size=(B, F)).astype(np.int32)
        cp, ct, cl, nc, nl = _expand(lp, flp, fc, k, width, base, base + F * k)
        for b in range(B):
            joint = []
            for f in range(F):
                top = np.argsort(-lp[b, f].astype(np.float64), kind="stable")[:k]
                sl = slice(base + f * k, base + (f + 1) * k)
                assert ct[b, sl].tolist() == top.tolist()
                assert (cp[b, sl] == fc[b, f]).all()
                want = (np.float32(flp[b, f]) + lp[b, f, top]).astype(np.float32)     # numpy's own fp32 addition
                assert np.array_equal(cl[b, sl], want)
                joint.extend(want.tolist())
            order = np.argsort(-np.asarray(joint, np.float64), kind="stable")[:width]
            assert nc[b].tolist() == (base + order).tolist()
            assert np.array_equal(nl[b], np.asarray(joint, np.float32)[order])


def test_levels_chained_into_the_builder_keep_path_sums():
    """Expand level by level, then build: every node's joint value is the fp32 sum along its path,
    and the joint values never grow along a path (log-probabilities are <= 0)."""
    B, V, k, width, levels, N = 2, 500, 4, 3, 4, 20
    cap = k + (levels - 1) * width * k
    cp = np.full((B, cap), -7, np.int32)
    ct = np.full((B, cap), -7, np.int32)
    cl = np.full((B, cap), np.nan, np.float32)
    fc = np.full((B, 1), -1, np.int32)
    flp = np.zeros((B, 1), np.float32)
    base = 0
    for lvl in range(levels):
        F = fc.shape[1]
        lp = synth.draft_logprob_rows(50 + lvl, B, F, V)
        fc, flp = oracle.draft_expand(lp, flp, fc, k, min(width, F * k), base, cp, ct, cl)
        base += F * k
    assert base == cap
    r = oracle.tree_build(cp, ct, cl, np.zeros(B, np.int32), N)
    assert r["valid"]
    for b in range(B):
        for c in range(cap):
            if cp[b, c] >= 0:
                assert cl[b, c] <= cl[b, cp[b, c]]
