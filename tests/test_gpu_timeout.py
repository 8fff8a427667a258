"""The bounded device-side wait and its route to the host: a wait on a barrier that nothing
arrives on runs out after its poll limit, the kernel returns, `fspad_status` reports
FSPAD_ERR_TIMEOUT once, and the context goes on working."""
import pytest
import torch

from paper_2408_15562_b200 import binding, synth
from tests import helpers

pytestmark = pytest.mark.gpu


def test_wait_runs_out_and_is_reported_once():
    w = synth.scaled(synth.WORKLOADS["llama3_8b_2k"], n_q_heads=8, n_kv_heads=2, prefix=(200, 200), n_nodes=12,
                     depth=3, branch=3, vocab=64, temperatures=(0.0,))
    inp = synth.generate(w, 0)
    ctx = helpers.make_ctx(inp)
    for polls in (1, 64, 1000):
        assert ctx.selftest_wait_timeout(polls) == 0
        assert ctx.status() == -7 and "wait" in binding.strerror(-7)
        assert ctx.status() == 0                      # cleared by the read
    assert ctx.selftest_wait_timeout(0) == -5 and ctx.selftest_wait_timeout(5000) == -5
    # the context is intact: an attention call afterwards is correct
    import oracle
    d = helpers.upload_attn(inp)
    out = ctx.tree_attn(d["q"], d["k_cache"], d["v_cache"], d["tree_k"], d["tree_v"], d["parent"], d["prefix_len"])
    ctx.check()
    ref = oracle.tree_attn(inp.q, inp.k_cache, inp.v_cache, inp.tree_k, inp.tree_v, inp.parent, inp.prefix_len)
    mx, mean = helpers.attn_errors(out, ref)
    assert mx <= 1e-2 and mean <= 1e-3
    torch.cuda.synchronize()
