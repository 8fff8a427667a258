"""The LM-head product with the scan as its epilogue (`fspad_lm_head_stats`, `fspad_lm_head_accept`)
against the oracle.

Tolerances (bf16 inputs, exact products, fp32 accumulation over H terms in H / 16 tensor-core steps):
a logit differs from the fp64 value by at most (H / 16) roundings of a running sum of magnitude <= 16,
i.e. 256 * 16 * 2^-24 = 2.4e-4 at H = 4096; LOGIT_TOL = 1e-3 leaves a factor of four.  The maximum
carries the same error; the argmax must be the oracle's wherever the oracle's maximum leads its
runner-up by more than 2 * LOGIT_TOL (rows with a smaller gap are counted); the sum of exponentials
inherits a relative error of LOGIT_TOL / T from its exponents plus the scan's own 2e-6.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth
from tests import helpers

pytestmark = pytest.mark.gpu

LOGIT_TOL = 1e-3


def _stats_case(seed, rows, H, V, rows_per_seq, temps, want_logits):
    h, w = synth.lm_head_inputs(seed, rows, H, V)
    ctx = binding.Context(8, 8, V, 128, max_nodes=rows_per_seq, max_batch=(rows + rows_per_seq - 1) // rows_per_seq)
    dh, dw = binding.bf16_tensor(h), binding.bf16_tensor(w)
    temperature = torch.tensor(temps, dtype=torch.float32, device="cuda")
    lg = torch.full((rows, V), float("nan"), dtype=torch.float32, device="cuda") if want_logits else None
    m, s, a = ctx.lm_head_stats(dh, dw, temperature, rows_per_seq, logits_out=lg)
    ctx.check()
    m, s, a = m.cpu().numpy(), s.cpu().numpy(), a.cpu().numpy()
    close_calls = 0
    for s0 in range(0, rows, rows_per_seq):
        T = float(temps[s0 // rows_per_seq]) or 1.0
        sl = slice(s0, min(rows, s0 + rows_per_seq))
        r = oracle.lm_head_stats(h[sl], w, T, want_logits=want_logits)
        np.testing.assert_allclose(m[sl], r["max"], rtol=0, atol=LOGIT_TOL)
        np.testing.assert_allclose(s[sl], r["sum"], rtol=2 * LOGIT_TOL / T + 1e-5)
        for i in range(sl.start, sl.stop):
            if r["gap"][i - s0] > 2 * LOGIT_TOL:
                assert a[i] == r["arg"][i - s0], (i, a[i], r["arg"][i - s0], r["gap"][i - s0])
            else:
                close_calls += 1
        if want_logits:
            got = lg[sl].cpu().numpy().astype(np.float64)
            assert np.isfinite(got).all()
            assert np.abs(got - r["logits"]).max() <= LOGIT_TOL
    return close_calls


@pytest.mark.parametrize("rows,H,V", [(60, 256, 1024), (5, 64, 300), (128, 512, 1281), (1, 4096, 640), (77, 136, 4099)])
def test_stats_small_shapes_ragged_tiles(rows, H, V):
    """Tiles of 128 vocabulary entries with a ragged last tile, hidden sizes that are not multiples of the
    64-element stage, more tiles than SMs and fewer, with and without the logits output."""
    rps = rows if rows < 20 else 20
    n_seq = (rows + rps - 1) // rps
    temps = [(1.0, 0.7, 0.0, 1.3)[i % 4] for i in range(n_seq)]
    assert _stats_case(1, rows, H, V, rps, temps, True) <= 1
    assert _stats_case(2, rows, H, V, rps, temps, False) <= 1


def test_stats_more_rows_than_one_slab():
    assert _stats_case(3, 300, 128, 2000, 60, [1.0, 0.5, 1.0, 2.0, 1.0], True) <= 2


def test_stats_headline_shape_sampled_rows():
    """60 rows x hidden 4096 x vocabulary 128256 (the launch configuration the benchmark times); the oracle
    checks a sample of the rows in full (fp64 product over the whole vocabulary)."""
    rows, H, V = 60, 4096, 128256
    h, w = synth.lm_head_inputs(0, rows, H, V)
    ctx = binding.Context(32, 8, V, 128, max_nodes=60, max_batch=1)
    dh, dw = binding.bf16_tensor(h), binding.bf16_tensor(w)
    temperature = torch.ones(1, dtype=torch.float32, device="cuda")
    lg = torch.empty((rows, V), dtype=torch.float32, device="cuda")
    m, s, a = ctx.lm_head_stats(dh, dw, temperature, 60, logits_out=lg)
    ctx.check()
    pick = [0, 17, 59]
    r = oracle.lm_head_stats(np.ascontiguousarray(h[pick]), w, 1.0, want_logits=True)
    np.testing.assert_allclose(m.cpu().numpy()[pick], r["max"], rtol=0, atol=LOGIT_TOL)
    np.testing.assert_allclose(s.cpu().numpy()[pick], r["sum"], rtol=2 * LOGIT_TOL + 1e-5)
    for k, i in enumerate(pick):
        assert r["gap"][k] <= 2 * LOGIT_TOL or int(a[i]) == int(r["arg"][k])
        assert np.abs(lg[i].cpu().numpy().astype(np.float64) - r["logits"][k]).max() <= LOGIT_TOL
    # every row: the statistics agree with the scan of the logits the same call wrote
    m2, s2, a2 = oracle.row_stats(lg.cpu().numpy(), 1.0)
    np.testing.assert_array_equal(m.cpu().numpy().astype(np.float64), m2)
    np.testing.assert_array_equal(a.cpu().numpy(), a2)
    np.testing.assert_allclose(s.cpu().numpy(), s2, rtol=2e-6)


@pytest.mark.parametrize("mode", ["greedy", "sample", "mixed"])
def test_accept_behind_the_lm_head(mode):
    """Acceptance fed by hidden states: the result must be the oracle's acceptance of the logits the call
    itself produced (written out for the sampling walk; for the all-greedy case they are produced by a
    second call that only writes logits), bit-exact as for fspad_tree_accept."""
    temps = {"greedy": (0.0, 0.0, 0.0), "sample": (1.0, 0.8, 1.0), "mixed": (0.0, 1.0, 0.0)}[mode]
    V, H = 4096, 256
    w0 = synth.scaled(synth.WORKLOADS["llama3_8b_2k"], batch=3, vocab=V, n_nodes=24, depth=4, branch=4, temperatures=temps,
                      prefix=(8, 8))
    inp = synth.generate(w0, 3, with_attention=False)
    B, N = inp.parent.shape
    h, w = synth.lm_head_inputs(5, B * N, H, V)
    ctx = binding.Context(8, 8, V, 128, max_nodes=N, max_batch=B)
    dh, dw = binding.bf16_tensor(h).view(B, N, H), binding.bf16_tensor(w)
    temperature = helpers.dev(inp.temperature)
    # the logits this product gives (GPU), then inputs that are consistent with them: draft distributions
    # and children drawn the way the workloads do it, from those logits
    lg = torch.empty((B, N, V), dtype=torch.float32, device="cuda")
    ctx.lm_head_stats(dh.view(B * N, H), dw, temperature, N, logits_out=lg.view(B * N, V))
    ctx.check()
    inp.target_logits = lg.cpu().numpy()
    rng = np.random.default_rng(11)
    sampling = mode != "greedy"
    if sampling:
        z = inp.target_logits.astype(np.float64) + rng.standard_normal(inp.target_logits.shape)
        q = np.exp(z - z.max(-1, keepdims=True))
        inp.draft_probs = (q / q.sum(-1, keepdims=True)).astype(np.float32)
    for b in range(B):
        for i, ch in enumerate(synth.children_lists(inp.parent[b])):
            if not ch:
                continue
            if inp.temperature[b] > 0:
                p = inp.draft_probs[b, i].astype(np.float64)
                inp.draft_tokens[b, ch] = rng.choice(V, size=len(ch), replace=False, p=p / p.sum())
            else:
                noisy = inp.target_logits[b, i] + rng.standard_normal(V).astype(np.float32)
                inp.draft_tokens[b, ch] = np.argsort(-noisy, kind="stable")[:len(ch)]
    d = helpers.upload_accept(inp)
    lg2 = torch.zeros_like(lg) if sampling else None
    path, n_acc, bonus = ctx.lm_head_accept(dh, dw, d["draft_probs"], d["draft_tokens"], d["parent"], d["temperature"],
                                            d["uniforms"], logits=lg2)
    ctx.check()
    if sampling:
        assert torch.equal(lg2, lg)                       # same product, same logits
    hard, near, msgs = helpers.compare_accept(inp, path.cpu().numpy(), n_acc.cpu().numpy(), bonus.cpu().numpy())
    assert hard == 0 and near == 0, msgs
