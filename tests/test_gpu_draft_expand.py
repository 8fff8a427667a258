"""CUDA draft step (through the C ABI) against the oracle: tokens, parents, joint values (one fp32
addition) and the next frontier, all bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _check(ctx, lp, flp, fc, k, width, base, cap):
    B = lp.shape[0]
    ref = [np.full((B, cap), -7, np.int32), np.full((B, cap), -7, np.int32), np.full((B, cap), -3.5, np.float32)]
    nc_ref, nl_ref = oracle.draft_expand(lp, flp, fc, k, width, base, *ref)
    got = [_dev(np.full((B, cap), -7, np.int32)), _dev(np.full((B, cap), -7, np.int32)),
           _dev(np.full((B, cap), -3.5, np.float32))]
    nc, nl = ctx.draft_expand(_dev(lp), _dev(flp), _dev(fc), k, width, base, *got)
    ctx.check()
    for g, r in zip(got, ref):
        assert np.array_equal(g.cpu().numpy(), r)            # new entries equal, all others untouched
    assert np.array_equal(nc.cpu().numpy(), nc_ref)
    assert np.array_equal(nl.cpu().numpy(), nl_ref)


@pytest.mark.parametrize("vocab", [17, 1000, 4099, 32000, 128256])
@pytest.mark.parametrize("step", [0.0, 0.5])
def test_vocab_sizes_and_ties(vocab, step):
    """Rows shorter than one piece, ragged last pieces, unaligned row starts (odd vocab), 32 pieces."""
    ctx = binding.Context(8, 2, vocab, 256, max_nodes=64, max_batch=4)
    rng = np.random.default_rng(vocab)
    for seed, (F, k, width) in enumerate([(1, 10, 10), (10, 10, 10), (16, 16, 16), (3, 5, 15)]):
        if k > vocab:
            continue
        B = 2
        lp = synth.draft_logprob_rows(seed, B, F, vocab, step=step)
        flp = (-rng.random((B, F)) * 4).astype(np.float32)
        fc = rng.integers(-1, 50, size=(B, F)).astype(np.int32)
        _check(ctx, lp, flp, fc, k, width, 50, 50 + F * k + 3)


def test_minus_infinity_rows_and_zero_values():
    vocab = 5000
    ctx = binding.Context(8, 2, vocab, 256, max_nodes=64, max_batch=2)
    lp = synth.draft_logprob_rows(1, 2, 4, vocab)
    lp[0, 0, :] = -np.inf                       # impossible everywhere: tokens 0 .. k-1 by index
    lp[0, 1, 10:] = -np.inf                     # fewer finite values than k
    lp[1, 2, 77] = 0.0
    lp[1, 2, 78] = -0.0                         # the two zeros are one value: the lower token first
    flp = np.zeros((2, 4), np.float32)
    fc = np.full((2, 4), -1, np.int32)
    _check(ctx, lp, flp, fc, 12, 7, 0, 48)


def test_whole_draft_phase_then_builder_matches_the_oracle_chain():
    """Five levels of top-10 expansion on the device, then the builder: the flattened 60-node tree
    equals the one the oracle derives from the same log-probability rows."""
    B, V, k, width, levels, N = 2, 32000, 10, 10, 5, 60
    cap = k + (levels - 1) * width * k
    ctx = binding.Context(8, 2, V, 256, max_nodes=N, max_batch=B)
    ref = [np.full((B, cap), -7, np.int32), np.full((B, cap), -7, np.int32), np.full((B, cap), 0, np.float32)]
    dev = [_dev(a.copy()) for a in ref]
    fc_r, fl_r = np.full((B, 1), -1, np.int32), np.zeros((B, 1), np.float32)
    fc_d, fl_d = _dev(fc_r), _dev(fl_r)
    base = 0
    for lvl in range(levels):
        F = fc_r.shape[1]
        lp = synth.draft_logprob_rows(300 + lvl, B, F, V)
        fc_r, fl_r = oracle.draft_expand(lp, fl_r, fc_r, k, min(width, F * k), base, *ref)
        fc_d, fl_d = ctx.draft_expand(_dev(lp), fl_d, fc_d, k, min(width, F * k), base, *dev)
        base += F * k
    root = np.array([5, 6], np.int32)
    want = oracle.tree_build(*ref, root, N)
    parent, token, cand, n_out = ctx.tree_build(*dev, _dev(root), N)
    ctx.check()
    assert want["valid"]
    assert np.array_equal(parent.cpu().numpy(), want["parent"])
    assert np.array_equal(token.cpu().numpy(), want["token"])
    assert np.array_equal(cand.cpu().numpy(), want["cand"])


def test_host_detected_errors():
    ctx = binding.Context(8, 2, 1000, 256, max_nodes=64, max_batch=1)
    lp = _dev(synth.draft_logprob_rows(0, 1, 2, 1000))
    args = (_dev(np.zeros((1, 2), np.float32)), _dev(np.full((1, 2), -1, np.int32)))
    arrs = [_dev(np.zeros((1, 8), np.int32)), _dev(np.zeros((1, 8), np.int32)), _dev(np.zeros((1, 8), np.float32))]
    with pytest.raises(binding.FspadError):
        ctx.draft_expand(lp, *args, 5, 4, 0, *arrs)          # 2 * 5 new candidates do not fit 8 entries
    with pytest.raises(binding.FspadError):
        ctx.draft_expand(lp, *args, 17, 4, 0, *arrs)         # top_k beyond 16
    with pytest.raises(binding.FspadError):
        ctx.draft_expand(lp, *args, 2, 5, 0, *arrs)          # width beyond the new candidates
