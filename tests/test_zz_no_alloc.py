"""The allocation-free variant of the per-node vocabulary scan.

`fspad_accept_stats_noalloc` is for programs that may not call cudaMalloc (a
server whose memory pool owns the device, a path that must not synchronise):
it needs no context and keeps its scratch in a fixed array of the library.
Checked here through the C ABI against the regular `fspad_accept_stats` and
against the fp64 oracle on two calls in a row with different inputs and shapes,
so that state left in the shared scratch array by the first call cannot leak
into the second; also at the edges of its fixed capacity (one row of the largest
vocabulary, which needs the most partial slots per row, and the 1024-row limit).
This file sorts last on purpose: a failure here stops nothing else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding

pytestmark = pytest.mark.gpu


def _both(rows, vocab, rows_per_seq, temps, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    logits = torch.randn((rows, vocab), generator=g, device="cuda", dtype=torch.float32) * 3
    logits[rows // 2, vocab // 3] = logits[rows // 2].max()          # a duplicated maximum
    logits[rows // 2, vocab // 3 + 5] = logits[rows // 2, vocab // 3]
    temperature = torch.tensor(temps, dtype=torch.float32, device="cuda")
    ctx = binding.Context(8, 8, vocab, 128, max_nodes=rows_per_seq, max_batch=rows // rows_per_seq)
    want = ctx.accept_stats(logits, temperature, rows_per_seq)
    ctx.check()
    out = (torch.full((rows,), -1.0, dtype=torch.float32, device="cuda"),
           torch.full((rows,), -1.0, dtype=torch.float64, device="cuda"),
           torch.full((rows,), -1, dtype=torch.int32, device="cuda"))
    rc = binding.accept_stats_noalloc(logits, temperature, rows_per_seq, out)
    assert rc == 0, binding.strerror(rc)
    torch.cuda.synchronize()
    assert torch.equal(out[0], want[0])                               # maxima: exact
    assert torch.equal(out[2], want[2])                               # argmax (lowest index): exact
    np.testing.assert_allclose(out[1].cpu().numpy(), want[1].cpu().numpy(), rtol=2e-6)
    # and against the oracle's definition of the three row statistics, row by row at its temperature
    lg = logits.cpu().numpy()
    for s0 in range(0, rows, rows_per_seq):
        T = float(temps[s0 // rows_per_seq]) or 1.0
        m, sm, a = oracle.row_stats(lg[s0:s0 + rows_per_seq], T)
        np.testing.assert_array_equal(out[0][s0:s0 + rows_per_seq].cpu().numpy().astype(np.float64), m)
        np.testing.assert_array_equal(out[2][s0:s0 + rows_per_seq].cpu().numpy(), a)
        np.testing.assert_allclose(out[1][s0:s0 + rows_per_seq].cpu().numpy(), sm, rtol=2e-6)


def test_matches_context_entry_point_on_two_calls_in_a_row():
    _both(rows=120, vocab=128256, rows_per_seq=60, temps=[1.0, 0.7], seed=1)
    _both(rows=26, vocab=32003, rows_per_seq=26, temps=[0.0], seed=2)     # fewer rows, odd vocab, other slicing


def test_edges_of_the_fixed_capacity():
    _both(rows=1, vocab=128256, rows_per_seq=1, temps=[1.0], seed=3)        # one row cut into the most pieces
    _both(rows=4, vocab=128256, rows_per_seq=2, temps=[0.5, 1.0], seed=4)
    _both(rows=1024, vocab=4000, rows_per_seq=64, temps=[1.0] * 16, seed=5)  # the row limit itself


def test_rejects_sizes_beyond_its_fixed_capacity():
    logits = torch.zeros((1025, 8), dtype=torch.float32, device="cuda")
    out = (torch.empty(1025, dtype=torch.float32, device="cuda"), torch.empty(1025, dtype=torch.float64, device="cuda"),
           torch.empty(1025, dtype=torch.int32, device="cuda"))
    rc = binding.accept_stats_noalloc(logits, None, 64, out)
    assert rc == -10 and "capacity" in binding.strerror(rc)
