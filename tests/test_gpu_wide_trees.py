"""The verify step on trees of more than 64 nodes (up to 256: several mask words per node) against the oracle:
attention within the stated bound, acceptance bit-exact, compaction bit-exact, and the whole step in one call."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth
from tests import helpers

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


def _attn_check(inp, alias=False):
    ctx = helpers.make_ctx(inp)
    d = helpers.upload_attn(inp)
    out = ctx.tree_attn(d["q"], d["k_cache"], d["v_cache"], None if alias else d["tree_k"], None if alias else d["tree_v"],
                        d["parent"], d["prefix_len"])
    ctx.check()
    ref = oracle.tree_attn(inp.q, inp.k_cache, inp.v_cache, inp.tree_k, inp.tree_v, inp.parent, inp.prefix_len)
    mx, mean = helpers.attn_errors(out, ref)
    assert mx <= 1e-2 and mean <= 1e-3, (mx, mean)


@pytest.mark.parametrize("tree,n", [("pruned", 65), ("pruned", 128), ("pruned", 200), ("bfs", 256), ("chain", 100), ("star", 129)])
@pytest.mark.parametrize("hq,hkv,prefix", [(8, 2, 300), (4, 4, 77)])
def test_attention(tree, n, hq, hkv, prefix):
    """Tree rows that span two or three 128-key chunks, masks of two to four words, one to eight row tiles."""
    w = synth.scaled(W["llama3_8b_2k"], n_q_heads=hq, n_kv_heads=hkv, prefix=(prefix, prefix), n_nodes=n, tree=tree,
                     depth=8, branch=10, vocab=16)
    _attn_check(synth.generate(w, 1, with_accept=False), alias=(n == 128))


def test_attention_bad_tree_is_reported():
    w = synth.scaled(W["llama3_8b_2k"], n_q_heads=8, n_kv_heads=2, prefix=(100, 100), n_nodes=150, depth=8, branch=10, vocab=16)
    inp = synth.generate(w, 0, with_accept=False)
    inp.parent[0, 140] = 145                       # a parent behind its child
    ctx = helpers.make_ctx(inp)
    d = helpers.upload_attn(inp)
    ctx.tree_attn(d["q"], d["k_cache"], d["v_cache"], d["tree_k"], d["tree_v"], d["parent"], d["prefix_len"])
    assert ctx.status() == -8


@pytest.mark.parametrize("n", [65, 130, 256])
@pytest.mark.parametrize("mode", ["greedy", "sample", "mixed"])
def test_acceptance(n, mode):
    temps = {"greedy": (0.0, 0.0), "sample": (1.0, 0.8), "mixed": (0.0, 1.0)}[mode]
    for vocab, variant in ((3000, 0), (32000, 1)):
        w = synth.scaled(W["llama3_8b_2k"], batch=2, vocab=vocab, n_nodes=n, depth=8, branch=10, temperatures=temps,
                         prefix=(8, 8))
        inp = synth.generate(w, variant, with_attention=False)
        ctx = helpers.make_ctx(inp)
        d = helpers.upload_accept(inp)
        path, n_acc, bonus = ctx.tree_accept(d["target_logits"], d["draft_probs"], d["draft_tokens"], d["parent"],
                                             d["temperature"], d["uniforms"])
        ctx.check()
        hard, near, msgs = helpers.compare_accept(inp, path.cpu().numpy(), n_acc.cpu().numpy(), bonus.cpu().numpy())
        assert hard == 0 and near == 0, msgs


def test_draft_far_from_target_on_a_wide_tree():
    """Many rejections per node (children of a node can number ten): the residual chain on the 256-node instance."""
    w = synth.scaled(W["llama3_8b_2k"], batch=4, vocab=2500, n_nodes=120, depth=5, branch=10, temperatures=(1.0,) * 4,
                     prefix=(8, 8))
    inp = synth.generate(w, 2, with_attention=False)
    rng = np.random.default_rng(3)
    z = rng.standard_normal(inp.draft_probs.shape) * 3
    q = np.exp(z - z.max(-1, keepdims=True))
    inp.draft_probs[...] = (q / q.sum(-1, keepdims=True)).astype(np.float32)
    for b in range(w.batch):
        for i, ch in enumerate(synth.children_lists(inp.parent[b])):
            if ch:
                inp.draft_tokens[b, ch] = np.argsort(-inp.draft_probs[b, i], kind="stable")[:len(ch)]
    ctx = helpers.make_ctx(inp)
    d = helpers.upload_accept(inp)
    path, n_acc, bonus = ctx.tree_accept(d["target_logits"], d["draft_probs"], d["draft_tokens"], d["parent"], d["temperature"],
                                         d["uniforms"])
    ctx.check()
    hard, near, msgs = helpers.compare_accept(inp, path.cpu().numpy(), n_acc.cpu().numpy(), bonus.cpu().numpy())
    assert hard == 0 and near == 0, msgs


def test_whole_step_with_200_nodes():
    w = synth.scaled(W["llama3_8b_2k"], batch=2, prefix=(150, 400), n_nodes=200, depth=8, branch=10, vocab=5000,
                     temperatures=(1.0, 0.0))
    inp = synth.generate(w, 4)
    B, N = inp.parent.shape
    cache_host = synth.make_cache(inp, 2)
    ref_o = oracle.tree_attn(inp.q, inp.k_cache, inp.v_cache, inp.tree_k, inp.tree_v, inp.parent, inp.prefix_len)
    r = oracle.tree_accept(inp.target_logits, inp.draft_probs, inp.draft_tokens, inp.parent, inp.temperature, inp.uniforms)
    want = cache_host.copy()
    want_len = oracle.kv_compact(want, r["accepted_path"], r["n_accepted"], inp.prefix_len)
    ctx = helpers.make_ctx(inp, n_layers=2)
    d, a = helpers.upload_accept(inp), helpers.upload_attn(inp)
    cache = binding.bf16_tensor(cache_host)
    out = torch.empty_like(a["q"])
    path = torch.full((B, N), -7, dtype=torch.int32, device="cuda")
    n_acc, bonus, new_len = (torch.empty((B,), dtype=torch.int32, device="cuda") for _ in range(3))
    ctx.verify_step(cache, a["q"], a["tree_k"], a["tree_v"], a["parent"], a["prefix_len"], d["target_logits"], d["draft_probs"],
                    d["draft_tokens"], d["temperature"], d["uniforms"], out, path, n_acc, bonus, new_len)
    ctx.check()
    mx, mean = helpers.attn_errors(out, ref_o)
    assert mx <= 1e-2 and mean <= 1e-3
    hard, near, msgs = helpers.compare_accept(inp, path.cpu().numpy(), n_acc.cpu().numpy(), bonus.cpu().numpy())
    assert hard == 0 and near == 0, msgs
    got = binding.bf16_bits(cache)
    for b in range(B):
        np.testing.assert_array_equal(got[:, :, b, :, :int(want_len[b])], want[:, :, b, :, :int(want_len[b])])
    np.testing.assert_array_equal(new_len.cpu().numpy(), want_len)


def test_limits():
    with pytest.raises(binding.FspadError) as e:
        binding.Context(8, 2, 100, 600, max_nodes=257)
    assert e.value.code == -4
    ctx = binding.Context(8, 2, 100, 600, max_nodes=256)
    cand = torch.zeros((1, 300), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.FspadError) as e:        # the tree builder keeps its 64-node limit
        ctx.tree_build(cand - 1, cand, torch.zeros((1, 300), dtype=torch.float32, device="cuda"),
                       torch.zeros(1, dtype=torch.int32, device="cuda"), 65)
    assert e.value.code == -4
