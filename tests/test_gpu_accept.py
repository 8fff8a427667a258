"""CUDA acceptance (through the C ABI) against the oracle: bit-exact path, length
and bonus token; divergences are tolerated only inside the 1e-6 decision band and
are counted."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import synth
from tests import helpers

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


def _run(inp, ctx=None):
    ctx = ctx or helpers.make_ctx(inp)
    d = helpers.upload_accept(inp)
    path, n_acc, bonus = ctx.tree_accept(d["target_logits"], d["draft_probs"], d["draft_tokens"], d["parent"],
                                         d["temperature"], d["uniforms"])
    ctx.check()
    return path.cpu().numpy(), n_acc.cpu().numpy(), bonus.cpu().numpy()


def _assert_parity(inp, allow_near=0):
    path, n_acc, bonus = _run(inp)
    hard, near, msgs = helpers.compare_accept(inp, path, n_acc, bonus)
    assert hard == 0, msgs
    assert near <= allow_near, msgs
    return near


@pytest.mark.parametrize("vocab", [8, 33, 1000, 4099, 32000])
@pytest.mark.parametrize("mode", ["greedy", "sample", "mixed"])
def test_small_trees_many_seeds(vocab, mode):
    temps = {"greedy": (0.0,) * 4, "sample": (1.0, 1.0, 0.7, 1.3), "mixed": (0.0, 1.0, 0.0, 0.5)}[mode]
    total_near = 0
    for variant in range(6):
        w = synth.scaled(W["llama3_8b_2k"], batch=4, vocab=vocab, n_nodes=min(20, vocab), depth=4, branch=3,
                         temperatures=temps, prefix=(8, 8))
        inp = synth.generate(w, variant, with_attention=False)
        total_near += _assert_parity(inp, allow_near=1)
    assert total_near <= 1


@pytest.mark.parametrize("tree", ["chain", "star", "bfs"])
def test_special_trees(tree):
    for temps in ((0.0, 0.0), (1.0, 1.0)):
        w = synth.scaled(W["tiny_greedy"], batch=2, vocab=2000, n_nodes=9, tree=tree, branch=2,
                         temperatures=temps, prefix=(8, 8))
        for variant in range(4):
            _assert_parity(synth.generate(w, variant, with_attention=False))


def test_root_only_tree_and_max_nodes():
    for n in (1, 64):
        w = synth.scaled(W["llama3_8b_2k"], batch=2, vocab=5000, n_nodes=n, depth=5 if n > 1 else 1, branch=4,
                         temperatures=(0.0, 1.0), prefix=(8, 8))
        _assert_parity(synth.generate(w, 0, with_attention=False))


def test_draft_far_from_target_forces_many_rejections():
    """A draft distribution unrelated to the target: most children are rejected,
    so the residual chain and the bonus draw from a deep residual are exercised."""
    w = synth.scaled(W["llama3_8b_2k"], batch=8, vocab=3000, n_nodes=24, depth=3, branch=8,
                     temperatures=(1.0,) * 8, prefix=(8, 8))
    rejected_somewhere = 0
    for variant in range(4):
        inp = synth.generate(w, variant, with_attention=False)
        rng = np.random.default_rng(variant)
        z = rng.standard_normal(inp.draft_probs.shape) * 3
        q = np.exp(z - z.max(-1, keepdims=True))
        inp.draft_probs[...] = (q / q.sum(-1, keepdims=True)).astype(np.float32)
        for b in range(w.batch):                    # children carry the draft's own favourite tokens
            for i, ch in enumerate(synth.children_lists(inp.parent[b])):
                if ch:
                    inp.draft_tokens[b, ch] = np.argsort(-inp.draft_probs[b, i], kind="stable")[:len(ch)]
        _assert_parity(inp)
        r = oracle.tree_accept(inp.target_logits, inp.draft_probs, inp.draft_tokens, inp.parent,
                               inp.temperature, inp.uniforms)
        rejected_somewhere += int((~np.isnan(r["trace_rq"])).sum() - (r["n_accepted"] - 1).sum())
    assert rejected_somewhere > 20


def test_draft_equal_to_target_up_to_fp32_rounding():
    """q = softmax(logits) up to a few fp32 ulps: every token sits inside the band where the scan's approximate
    denominator cannot fix the sign of p - q, so the one-sweep first rejection must hand over to the
    exact two-sweep path; the residual mass itself is of the order of fp32 rounding."""
    w = synth.scaled(W["llama3_8b_2k"], batch=6, vocab=5000, n_nodes=24, depth=3, branch=8,
                     temperatures=(1.0, 1.0, 0.7, 0.7, 1.3, 1.3), prefix=(8, 8))
    rejected = 0
    for variant in range(3):
        inp = synth.generate(w, variant, with_attention=False)
        z = inp.target_logits.astype(np.float64) / inp.temperature[:, None, None].astype(np.float64)
        p = np.exp(z - z.max(-1, keepdims=True))
        wobble = 1.0 + 3e-7 * np.random.default_rng(variant).choice([-1.0, 1.0], size=p.shape)
        inp.draft_probs[...] = (p / p.sum(-1, keepdims=True) * wobble).astype(np.float32)
        # uniforms just below one: r * q < p now fails wherever q lies above p, so rejections do occur
        keep = inp.uniforms[:, -1].copy()
        inp.uniforms[...] = np.nextafter(np.float32(1), np.float32(0))
        inp.uniforms[:, -1] = keep
        _assert_parity(inp, allow_near=w.batch)
        r = oracle.tree_accept(inp.target_logits, inp.draft_probs, inp.draft_tokens, inp.parent,
                               inp.temperature, inp.uniforms)
        rejected += int((~np.isnan(r["trace_rq"])).sum() - (r["n_accepted"] - 1).sum())
    assert rejected > 0


def test_zero_mass_and_minus_inf_logits():
    w = synth.scaled(W["llama3_8b_2k"], batch=4, vocab=512, n_nodes=16, depth=4, branch=3,
                     temperatures=(1.0,) * 4, prefix=(8, 8))
    inp = synth.generate(w, 3, with_attention=False)
    rng = np.random.default_rng(0)
    kill = rng.random(inp.target_logits.shape) < 0.3
    inp.target_logits[kill] = -np.inf
    dz = rng.random(inp.draft_probs.shape) < 0.3
    inp.draft_probs[dz] = 0.0
    _assert_parity(inp)


def test_stats_pass_matches_oracle_rows():
    w = synth.scaled(W["llama3_8b_2k"], batch=2, vocab=128256, n_nodes=7, depth=3, branch=3,
                     temperatures=(1.0, 0.6), prefix=(8, 8))
    inp = synth.generate(w, 0, with_attention=False)
    inp.target_logits[0, 3, 777] = inp.target_logits[0, 3].max()      # duplicate maxima: lowest index wins
    inp.target_logits[0, 3, 100000] = inp.target_logits[0, 3, 777]
    ctx = helpers.make_ctx(inp)
    lg = helpers.dev(inp.target_logits.reshape(-1, w.vocab))
    m, s, a = ctx.accept_stats(lg, helpers.dev(inp.temperature), 7)
    ctx.check()
    for b in range(2):
        om, os_, oa = oracle.row_stats(inp.target_logits[b], float(inp.temperature[b]))
        sl = slice(b * 7, b * 7 + 7)
        np.testing.assert_array_equal(m[sl].cpu().numpy().astype(np.float64), om)
        np.testing.assert_array_equal(a[sl].cpu().numpy(), oa)
        np.testing.assert_allclose(s[sl].cpu().numpy(), os_, rtol=2e-6)
    assert int(a[3]) == min(777, int(np.argmax(inp.target_logits[0, 3])))


@pytest.mark.parametrize("name", ["tiny_greedy", "llama3_8b_2k", "vicuna_33b_4k_greedy",
                                  "vicuna_33b_4k_sample", "llama3_70b_8k"])
def test_full_size_single_sequence_configs(name):
    for variant in range(2):
        inp = synth.generate(W[name], variant, with_attention=False)
        _assert_parity(inp, allow_near=1)


def test_full_size_batch16_mixed():
    inp = synth.generate(W["batch16_ragged"], 0, with_attention=False)
    _assert_parity(inp, allow_near=1)


def test_device_detected_errors_are_reported_not_fatal():
    w = synth.scaled(W["tiny_greedy"], vocab=1000, n_nodes=8, prefix=(8, 8))
    inp = synth.generate(w, 0, with_attention=False)
    ctx = helpers.make_ctx(inp)
    bad = inp.parent.copy()
    bad[0, 3] = 5                                   # parent after child
    d = helpers.upload_accept(inp)
    ctx.tree_accept(d["target_logits"], None, d["draft_tokens"], helpers.dev(bad), d["temperature"], None)
    assert ctx.status() == -8
    assert ctx.status() == 0                        # cleared by the read
    toks = inp.draft_tokens.copy()
    toks[0, 2] = 1000                               # token id == V
    ctx.tree_accept(d["target_logits"], None, helpers.dev(toks), d["parent"], d["temperature"], None)
    assert ctx.status() == -5
    # the context still works
    path, n_acc, bonus = _run(inp, ctx)
    assert helpers.compare_accept(inp, path, n_acc, bonus)[0] == 0
