"""The host-buffer entry point (`fspad_verify_step_host`) against the oracle (attention within the
stated bound, acceptance and compacted cache bit-exact) and against the three device calls it
stands for: same attention output, same acceptance result, same compacted cache, twice in a row."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth
from tests import helpers

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


@pytest.mark.parametrize("mode", ["sample", "greedy", "mixed"])
def test_host_entry_equals_device_calls(mode):
    temps = {"sample": (1.0, 0.8, 1.0), "greedy": (0.0, 0.0, 0.0), "mixed": (0.0, 1.0, 0.0)}[mode]
    w = synth.scaled(W["llama3_8b_2k"], batch=3, prefix=(40, 300), n_nodes=24, depth=4, branch=4, vocab=3000,
                     temperatures=temps)
    inp = synth.generate(w, 5)
    B, N = inp.parent.shape
    ctx = helpers.make_ctx(inp, n_layers=2)
    cache_host = synth.make_cache(inp, 2)
    L = inp.prefix_len
    for b in range(B):                          # the device path takes the tree rows from the cache
        cache_host[0, 0, b, :, L[b]:L[b] + N] = inp.tree_k[b]
        cache_host[0, 1, b, :, L[b]:L[b] + N] = inp.tree_v[b]
    # --- device calls ---
    cache_d = binding.bf16_tensor(cache_host)
    d = helpers.upload_accept(inp)
    parent, prefix = helpers.dev(inp.parent), helpers.dev(inp.prefix_len)
    out_d = ctx.tree_attn(binding.bf16_tensor(inp.q), cache_d[0, 0], cache_d[0, 1], None, None, parent, prefix)
    path_d, n_d, bonus_d = ctx.tree_accept(d["target_logits"], d["draft_probs"], d["draft_tokens"], parent,
                                           d["temperature"], d["uniforms"])
    len_d = ctx.kv_compact(cache_d, path_d, n_d, prefix)
    ctx.check()
    # --- the oracle on the same inputs ---
    ref_o = oracle.tree_attn(inp.q, inp.k_cache, inp.v_cache, inp.tree_k, inp.tree_v, inp.parent, inp.prefix_len)
    r = oracle.tree_accept(inp.target_logits, inp.draft_probs, inp.draft_tokens, inp.parent, inp.temperature,
                           inp.uniforms if inp.draft_probs is not None else None)
    want_cache = cache_host.copy()
    want_len = oracle.kv_compact(want_cache, r["accepted_path"], r["n_accepted"], inp.prefix_len)
    # --- host entry, two calls in a row on fresh caches ---
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()   # noqa: E731
    hq = binding.bf16_tensor(inp.q, "cpu").pin_memory()
    htk = binding.bf16_tensor(inp.tree_k, "cpu").pin_memory()
    htv = binding.bf16_tensor(inp.tree_v, "cpu").pin_memory()
    sampling = inp.draft_probs is not None
    for _ in range(2):
        cache_h = binding.bf16_tensor(synth.make_cache(inp, 2))      # tree rows come through the call
        hout = torch.empty_like(hq).pin_memory()
        hpath = torch.empty((B, N), dtype=torch.int32).pin_memory()
        hn, hb, hl = (torch.empty((B,), dtype=torch.int32).pin_memory() for _ in range(3))
        ctx.verify_step_host(cache_h, hq, htk, htv, pin(inp.parent), pin(inp.prefix_len), pin(inp.target_logits),
                             pin(inp.draft_probs) if sampling else None, pin(inp.draft_tokens), pin(inp.temperature),
                             pin(inp.uniforms) if sampling else None, hout, hpath, hn, hb, hl)
        torch.cuda.synchronize()
        mx, mean = helpers.attn_errors(hout, ref_o)
        assert mx <= 1e-2 and mean <= 1e-3, (mx, mean)
        hard, near, msgs = helpers.compare_accept(inp, hpath.numpy(), hn.numpy(), hb.numpy())
        assert hard == 0 and near == 0, msgs
        np.testing.assert_array_equal(hl.numpy(), want_len)
        got = binding.bf16_bits(cache_h)
        for b in range(B):
            np.testing.assert_array_equal(got[:, :, b, :, :int(want_len[b])], want_cache[:, :, b, :, :int(want_len[b])])
        assert torch.equal(hout.view(torch.int16), out_d.cpu().view(torch.int16))
        assert torch.equal(hn, n_d.cpu()) and torch.equal(hb, bonus_d.cpu()) and torch.equal(hl, len_d.cpu())
        for b in range(B):
            k = int(hn[b])
            assert torch.equal(hpath[b, :k], path_d[b, :k].cpu())
            rows = int(hl[b])
            assert torch.equal(cache_h[:, :, b, :, :rows].view(torch.int16), cache_d[:, :, b, :, :rows].view(torch.int16))
