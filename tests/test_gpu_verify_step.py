"""The whole verify step in one call (`fspad_verify_step`: attention on the context's second
stream beside acceptance, then compaction) against the oracle: attention within the stated bound,
acceptance and the compacted cache bit-exact.  Both forms of the tree rows (explicit arrays, and
rows of the cache that the compaction then rewrites), eager and replayed from a CUDA graph."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth
from tests import helpers

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


def _oracle_step(inp, cache_host, layer):
    ref_o = oracle.tree_attn(inp.q, inp.k_cache, inp.v_cache, inp.tree_k, inp.tree_v, inp.parent, inp.prefix_len)
    r = oracle.tree_accept(inp.target_logits, inp.draft_probs, inp.draft_tokens, inp.parent, inp.temperature,
                           inp.uniforms if inp.draft_probs is not None else None)
    want = cache_host.copy()
    want_len = oracle.kv_compact(want, r["accepted_path"], r["n_accepted"], inp.prefix_len)
    return ref_o, r, want, want_len


def _device_inputs(inp, cache_host):
    d = helpers.upload_accept(inp)
    a = helpers.upload_attn(inp)
    B, N = inp.parent.shape
    outs = dict(attn_out=torch.empty_like(a["q"]), path=torch.full((B, N), -7, dtype=torch.int32, device="cuda"),
                n_acc=torch.empty((B,), dtype=torch.int32, device="cuda"),
                bonus=torch.empty((B,), dtype=torch.int32, device="cuda"),
                new_len=torch.empty((B,), dtype=torch.int32, device="cuda"))
    return d, a, outs, binding.bf16_tensor(cache_host)


def _call(ctx, cache, a, d, outs, aliased, layer):
    ctx.verify_step(cache, a["q"], None if aliased else a["tree_k"], None if aliased else a["tree_v"], a["parent"],
                    a["prefix_len"], d["target_logits"], d["draft_probs"], d["draft_tokens"], d["temperature"],
                    d["uniforms"], outs["attn_out"], outs["path"], outs["n_acc"], outs["bonus"], outs["new_len"],
                    attn_layer=layer)


def _check(inp, outs, cache, ref_o, r, want, want_len):
    mx, mean = helpers.attn_errors(outs["attn_out"], ref_o)
    assert mx <= 1e-2 and mean <= 1e-3, (mx, mean)
    hard, near, msgs = helpers.compare_accept(inp, outs["path"].cpu().numpy(), outs["n_acc"].cpu().numpy(),
                                              outs["bonus"].cpu().numpy())
    assert hard == 0 and near == 0, msgs
    np.testing.assert_array_equal(outs["new_len"].cpu().numpy(), want_len)
    got = binding.bf16_bits(cache)
    for b in range(inp.parent.shape[0]):           # rows past the new length are dead
        rows = int(want_len[b])
        np.testing.assert_array_equal(got[:, :, b, :, :rows], want[:, :, b, :, :rows])


@pytest.mark.parametrize("n_layers", [3, 5])      # 48 and 80 (layer, K/V, head) slices per sequence: up to 64 the walk's
@pytest.mark.parametrize("aliased", [False, True])  # own CTAs compact the cache, above that the compaction kernel does
@pytest.mark.parametrize("mode", ["sample", "greedy", "mixed"])
def test_whole_step_against_oracle(mode, aliased, n_layers):
    temps = {"sample": (1.0, 0.8, 1.0), "greedy": (0.0, 0.0, 0.0), "mixed": (0.0, 1.0, 0.0)}[mode]
    w = synth.scaled(W["llama3_8b_2k"], batch=3, prefix=(40, 300), n_nodes=24, depth=4, branch=4, vocab=3000,
                     temperatures=temps)
    inp = synth.generate(w, 11)
    B, N = inp.parent.shape
    layer = 1
    cache_host = synth.make_cache(inp, n_layers)
    L = inp.prefix_len
    for b in range(B):          # the attention layer's planes are the workload's K/V; tree rows behind the prefix
        cache_host[layer, 0, b] = inp.k_cache[b]
        cache_host[layer, 1, b] = inp.v_cache[b]
        cache_host[layer, 0, b, :, L[b]:L[b] + N] = inp.tree_k[b]
        cache_host[layer, 1, b, :, L[b]:L[b] + N] = inp.tree_v[b]
    ref_o, r, want, want_len = _oracle_step(inp, cache_host, layer)
    ctx = helpers.make_ctx(inp, n_layers=n_layers)
    d, a, outs, cache = _device_inputs(inp, cache_host)
    _call(ctx, cache, a, d, outs, aliased, layer)
    ctx.check()
    _check(inp, outs, cache, ref_o, r, want, want_len)


def test_whole_step_headline_shape_in_a_graph():
    """Full llama3_8b_2k launch configuration, captured once and replayed: the fork and join of the
    second stream are part of the graph."""
    inp = synth.generate(W["llama3_8b_2k"], 0)
    cache_host = synth.make_cache(inp, 1)
    ref_o, r, want, want_len = _oracle_step(inp, cache_host, 0)
    ctx = helpers.make_ctx(inp, n_layers=1)
    d, a, outs, cache = _device_inputs(inp, cache_host)
    _call(ctx, cache, a, d, outs, False, 0)        # warm-up outside the capture (one-time attribute calls)
    torch.cuda.synchronize()
    cache.copy_(binding.bf16_tensor(cache_host))
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        _call(ctx, cache, a, d, outs, False, 0)
    outs["attn_out"].zero_()
    outs["path"].fill_(-7)
    g.replay()
    torch.cuda.synchronize()
    ctx.check()
    _check(inp, outs, cache, ref_o, r, want, want_len)


def test_argument_errors():
    w = synth.scaled(W["llama3_8b_2k"], batch=1, prefix=(40, 40), n_nodes=8, depth=3, branch=3, vocab=100,
                     temperatures=(0.0,))
    inp = synth.generate(w, 0)
    ctx = helpers.make_ctx(inp, n_layers=1)
    d, a, outs, cache = _device_inputs(inp, synth.make_cache(inp, 1))
    with pytest.raises(binding.FspadError) as e:
        _call(ctx, cache, a, d, outs, False, 1)    # layer out of range
    assert e.value.code == -3
    with pytest.raises(binding.FspadError) as e:
        ctx.verify_step(None, a["q"], None, None, a["parent"], a["prefix_len"], d["target_logits"], None,
                        d["draft_tokens"], d["temperature"], None, outs["attn_out"], outs["path"], outs["n_acc"],
                        outs["bonus"], outs["new_len"])
    assert e.value.code == -1
    _call(ctx, cache, a, d, outs, True, 0)         # and the context still works
    ctx.check()
