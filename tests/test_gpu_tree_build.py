"""CUDA tree builder (through the C ABI) against the oracle: integer outputs, bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _ctx(max_nodes=64, max_batch=16):
    return binding.Context(8, 2, 64, 256, max_nodes=max_nodes, max_batch=max_batch)


def _run(ctx, cp, ct, lp, rt, n):
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    anc = torch.empty((cp.shape[0], n), dtype=torch.int64, device="cuda")
    parent, token, cand, n_out = ctx.tree_build(dev(cp), dev(ct), dev(lp), dev(rt), n, anc=anc)
    return [t.cpu().numpy() for t in (parent, token, cand, n_out)] + [anc.cpu().numpy().view(np.uint64)]


def _assert_equal(ctx, cp, ct, lp, rt, n):
    ref = oracle.tree_build(cp, ct, lp, rt, n)
    assert ref["valid"]
    parent, token, cand, n_out, anc = _run(ctx, cp, ct, lp, rt, n)
    ctx.check()
    assert np.array_equal(anc, ref["anc"])
    assert np.array_equal(n_out, ref["n_out"])
    assert np.array_equal(parent, ref["parent"])
    assert np.array_equal(token, ref["token"])
    assert np.array_equal(cand, ref["cand"])


@pytest.mark.parametrize("step", [0.0, 0.5, 2.0])
@pytest.mark.parametrize("n_nodes", [1, 2, 30, 60, 64])
def test_paper_sized_candidate_lists(step, n_nodes):
    """410 candidates (top-10, five levels) down to 60 / 30 nodes (the paper's and the halved budget),
    with and without heavy ties."""
    ctx = _ctx()
    for seed in range(3):
        cp, ct, lp, rt = synth.tree_candidates(seed, 4, step=step)
        _assert_equal(ctx, cp, ct, lp, rt, n_nodes)


@pytest.mark.parametrize("levels,width,branch", [(1, 1, 1), (2, 1, 3), (3, 3, 5), (6, 12, 14), (9, 14, 9)])
def test_sizes_across_sorting_network_widths(levels, width, branch):
    """Candidate counts 1, 6, 35, 854, 972: sorting networks of 2, 8, 64 and 1024 entries, ragged."""
    ctx = _ctx()
    cp, ct, lp, rt = synth.tree_candidates(7, 3, levels=levels, width=width, branch=branch, vocab=128256, step=0.25)
    assert cp.shape[1] <= 1024
    for n in (5, 64):
        _assert_equal(ctx, cp, ct, lp, rt, n)


def test_minus_infinity_and_identical_values():
    ctx = _ctx()
    cp, ct, lp, rt = synth.tree_candidates(3, 2, levels=3, width=4, branch=4)
    lp[0, :] = -np.inf                      # every path impossible: order decided by index alone
    lp[1, :] = -1.0
    _assert_equal(ctx, cp, ct, lp, rt, 20)


def test_output_feeds_the_verification_step():
    """The flattened tree is a valid input of the acceptance call (topological parents)."""
    ctx = binding.Context(8, 2, 1000, 256, max_nodes=60, max_batch=2)
    cp, ct, lp, rt = synth.tree_candidates(11, 2, vocab=1000)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    parent, token, cand, n_out = ctx.tree_build(dev(cp), dev(ct), dev(lp), dev(rt), 60)
    logits = torch.randn(2, 60, 1000, device="cuda")
    temp = torch.zeros(2, device="cuda")
    path, n_acc, bonus = ctx.tree_accept(logits, None, token, parent, temp, None)
    ctx.check()
    assert (n_acc.cpu().numpy() >= 1).all()


def test_growing_probability_is_reported_not_fatal():
    ctx = _ctx()
    cp = np.array([[-1, 0, -1]], np.int32)
    lp = np.log(np.array([[0.1, 0.5, 0.3]], np.float32))
    _run(ctx, cp, np.array([[1, 2, 3]], np.int32), lp, np.array([0], np.int32), 3)
    assert ctx.status() == -8
    cp = np.array([[-1, 5, 0]], np.int32)    # parent index not below its own
    _run(ctx, cp, np.array([[1, 2, 3]], np.int32), lp, np.array([0], np.int32), 3)
    assert ctx.status() == -8


def test_host_detected_errors():
    ctx = _ctx(max_nodes=16)
    cp, ct, lp, rt = synth.tree_candidates(0, 1, levels=2, width=2, branch=2)
    with pytest.raises(binding.FspadError):
        _run(ctx, cp, ct, lp, rt, 17)        # beyond the context's max_nodes
