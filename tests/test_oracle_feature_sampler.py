"""Pins for the oracle's Feature Sampler forward (`oracle_feature_sampler`).

 * numpy float64 restatement with library matrix products and the logistic function from scipy
 * hand-worked 1 x 1 and 2 x 2 cases with exactly representable inputs (SiLU pinned at g = ln 3: 0.75 ln 3)
 * a zero Gate projector, or a zero Down projector, leaves the residual: eta == f exactly
 * doubling the Up projector doubles eta - f; negating the Gate input changes silu(g) to silu(-g) = silu(g) - g
 * rows are independent: permuting the rows permutes the outputs
"""
import numpy as np
from scipy.special import expit

import oracle
from paper_2408_15562_b200 import synth


def _f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def _b(a):
    return synth.f32_to_bf16_bits(np.asarray(a, np.float32))


def test_numpy_restatement():
    for seed, (R, H, I) in enumerate([(3, 32, 80), (7, 64, 40), (1, 8, 8)]):
        f, e, wu, wg, wd = synth.feature_sampler_inputs(seed, R, H, I)
        eta, s = oracle.feature_sampler(f, e, wu, wg, wd, want_inter=True)
        u = _f64(f) @ _f64(wu).T
        g = _f64(e) @ _f64(wg).T
        s_np = g * expit(g) * u
        np.testing.assert_allclose(s, s_np, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(eta, s_np @ _f64(wd).T + _f64(f), rtol=1e-12, atol=1e-13)


def test_hand_cases():
    # 1 x 1: f = 2, e = 1, Wup = 1.5, Wgate = 0 -> s = 0 -> eta = f
    assert oracle.feature_sampler(_b([[2.0]]), _b([[1.0]]), _b([[1.5]]), _b([[0.0]]), _b([[3.0]]))[0, 0] == 2.0
    # g = ln 3 is not exact in bf16, so pin SiLU through its bf16 value: silu(g) = g / (1 + exp(-g))
    gb = _b([[np.log(3.0)]])
    g = _f64(gb)[0, 0]
    eta = oracle.feature_sampler(_b([[2.0]]), _b([[1.0]]), _b([[1.5]]), gb, _b([[0.5]]))
    want = 0.5 * (g / (1 + np.exp(-g)) * 3.0) + 2.0
    assert abs(eta[0, 0] - want) < 1e-15 and abs(want - (0.5 * 0.75 * np.log(3) * 3 + 2)) < 0.01
    # 2 x 2 with a Down projector that swaps the two intermediate entries
    f, e = _b([[1.0, -2.0]]), _b([[0.5, 4.0]])
    wu, wg, wd = _b([[1, 0], [0, 1]]), _b([[2, 0], [0, 0.25]]), _b([[0, 1], [1, 0]])
    silu1 = 1.0 / (1 + np.exp(-1.0))                       # g = (1, 1): silu(1)
    eta = oracle.feature_sampler(f, e, wu, wg, wd)
    np.testing.assert_allclose(eta, [[silu1 * -2.0 + 1.0, silu1 * 1.0 - 2.0]], rtol=1e-15)


def test_zero_projectors_leave_the_residual():
    f, e, wu, wg, wd = synth.feature_sampler_inputs(5, 4, 48, 96)
    np.testing.assert_array_equal(oracle.feature_sampler(f, e, wu, np.zeros_like(wg), wd), _f64(f))
    np.testing.assert_array_equal(oracle.feature_sampler(f, e, wu, wg, np.zeros_like(wd)), _f64(f))


def test_scaling_symmetry_and_row_independence():
    f, e, wu, wg, wd = synth.feature_sampler_inputs(6, 5, 40, 72)
    eta, s = oracle.feature_sampler(f, e, wu, wg, wd, want_inter=True)
    wu2 = wu.copy()
    nz = wu2 & 0x7FFF != 0
    wu2[nz] += np.uint16(1 << 7)                           # every Up weight doubled, exactly
    eta2 = oracle.feature_sampler(f, e, wu2, wg, wd)
    np.testing.assert_allclose(eta2 - _f64(f), 2 * (eta - _f64(f)), rtol=1e-12, atol=1e-13)
    e_neg = e ^ np.uint16(0x8000)                          # e -> -e: g -> -g, silu(-g) = silu(g) - g
    _, s_neg = oracle.feature_sampler(f, e_neg, wu, wg, wd, want_inter=True)
    g = _f64(e) @ _f64(wg).T
    u = _f64(f) @ _f64(wu).T
    np.testing.assert_allclose(s_neg, s - g * u, rtol=1e-11, atol=1e-13)
    perm = np.array([3, 0, 4, 1, 2])
    eta_p = oracle.feature_sampler(np.ascontiguousarray(f[perm]), np.ascontiguousarray(e[perm]), wu, wg, wd)
    np.testing.assert_array_equal(eta_p, eta[perm])
