"""The Feature Sampler forward (`fspad_feature_sampler`) against the fp64 oracle.

Tolerance, from the arithmetic (bf16 operands, exact products, fp32 accumulation, bf16 results):
 * gated product s = silu(g) * u: g and u carry about 1e-5 of accumulation error, the result is rounded to
   bf16 (half an ulp = 2^-9 relative): |s_cuda - s| <= 2^-8 |s| + 1e-3;
 * eta = Wdown s + f: the Down product sees s rounded to bf16, I independent relative errors of 2^-9 whose
   sum has a standard deviation of about 2^-9 * rms(eta - f) (1.4e-3 for order-one values), and eta itself
   is rounded to bf16 (up to 2^-7 = 7.8e-3 absolute for |eta| in [2, 4)): max abs error <= 2.5e-2 and mean abs
   error <= 3e-3 for the order-one values the generator produces.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15562_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _check(seed, rows, H, I):
    f, e, wu, wg, wd = synth.feature_sampler_inputs(seed, rows, H, I)
    ctx = binding.Context(8, 8, 1000, 128, max_nodes=16, max_batch=1)
    d = [binding.bf16_tensor(x) for x in (f, e, wu, wg, wd)]
    eta, inter = ctx.feature_sampler(*d)
    ctx.check()
    want_eta, want_s = oracle.feature_sampler(f, e, wu, wg, wd, want_inter=True)
    got_s = inter.float().cpu().numpy().astype(np.float64)
    got_eta = eta.float().cpu().numpy().astype(np.float64)
    assert (np.abs(got_s - want_s) <= 2.0 ** -8 * np.abs(want_s) + 1e-3).all(), np.abs(got_s - want_s).max()
    err = np.abs(got_eta - want_eta)
    assert err.max() <= 2.5e-2 and err.mean() <= 3e-3, (err.max(), err.mean())
    return err.max(), err.mean()


@pytest.mark.parametrize("rows,H,I", [(10, 256, 704), (1, 64, 136), (60, 512, 1408), (128, 128, 264), (7, 1000, 40)])
def test_small_shapes(rows, H, I):
    """Sizes that are not multiples of the 128-column tile or the 64-element stage, one row and a full slab."""
    _check(1, rows, H, I)


def test_llama3_8b_shape_frontier_of_ten():
    """hidden 4096, intermediate 14336 (the intermediate_size of the 8B target), ten frontier rows: the
    launch configuration the benchmark times (three split products over all SMs)."""
    _check(2, 10, 4096, 14336)


def test_sixty_rows_and_argument_errors():
    _check(3, 60, 4096, 14336)
    ctx = binding.Context(8, 8, 1000, 128, max_nodes=16, max_batch=1)
    f, e, wu, wg, wd = synth.feature_sampler_inputs(0, 4, 64, 128)
    d = [binding.bf16_tensor(x) for x in (f, e, wu, wg, wd)]
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.FspadError) as ex:
        ctx.feature_sampler(*d, workspace=small)
    assert ex.value.code == -5
    big = [binding.bf16_tensor(x) for x in synth.feature_sampler_inputs(0, 129, 64, 128)]
    with pytest.raises(binding.FspadError) as ex:
        ctx.feature_sampler(*big)
    assert ex.value.code == -3
    ctx.feature_sampler(*d)
    ctx.check()
