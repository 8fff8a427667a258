"""Pins for the oracle's LM head + row statistics (`oracle_lm_head_stats`).

 * the logits equal numpy's float64 matrix product of the exactly converted bf16 inputs
 * a one-hot vocabulary matrix copies hidden columns: the statistics are those of the hidden
   row itself (values exact, ties resolved toward the lowest index)
 * hand-worked 2 x 3 case
 * scaling the hidden states by two doubles every logit: same argmax, doubled maximum and gap
 * permuting the vocabulary permutes the argmax and leaves maximum, sum and gap alone
 * its statistics agree with the existing row-statistics oracle run on its own logits
"""
import numpy as np

import oracle
from paper_2408_15562_b200 import synth


def _f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def test_logits_are_the_float64_matrix_product():
    for seed, (R, H, V) in enumerate([(5, 64, 97), (3, 257, 1000), (1, 16, 8)]):
        h, w = synth.lm_head_inputs(seed, R, H, V)
        for T in (1.0, 0.7):
            r = oracle.lm_head_stats(h, w, T, want_logits=True)
            z = _f64(h) @ _f64(w).T
            np.testing.assert_allclose(r["logits"], z, rtol=0, atol=1e-12 * np.abs(z).max())
            np.testing.assert_array_equal(r["arg"], np.argmax(r["logits"], axis=1))
            np.testing.assert_allclose(r["max"], r["logits"].max(axis=1), rtol=0, atol=0)
            np.testing.assert_allclose(r["sum"], np.exp((r["logits"] - r["max"][:, None]) / T).sum(axis=1), rtol=1e-13)
            srt = np.sort(r["logits"], axis=1)
            np.testing.assert_allclose(r["gap"], srt[:, -1] - srt[:, -2], rtol=0, atol=0)


def test_one_hot_vocabulary_matrix_copies_hidden_columns():
    rng = np.random.default_rng(3)
    R, H = 4, 12
    h = synth.normal_bf16(rng, (R, H))
    h[1, 7] = h[1, 2] = synth.f32_to_bf16_bits(np.array([5.0], np.float32))[0]    # a tie: columns 2 and 7
    cols = np.array([3, 7, 2, 0, 11, 5], np.int64)                                  # vocabulary entry v reads hidden column cols[v]
    w = np.zeros((len(cols), H), np.uint16)
    one = synth.f32_to_bf16_bits(np.array([1.0], np.float32))[0]
    w[np.arange(len(cols)), cols] = one
    r = oracle.lm_head_stats(h, w, 1.0, want_logits=True)
    x = _f64(h)[:, cols]
    np.testing.assert_array_equal(r["logits"], x)
    np.testing.assert_array_equal(r["max"], x.max(axis=1))
    assert r["arg"][1] == 1 and r["gap"][1] == 0.0       # 5.0 appears at vocabulary entries 1 (column 7) and 2 (column 2)
    np.testing.assert_array_equal(r["arg"], np.argmax(x, axis=1))


def test_hand_worked_case():
    # hidden = [[1, 2], [-1, 0.5]], weight rows = [1, 0], [0.5, 0.5], [-1, 1]  (all exact in bf16)
    b = lambda a: synth.f32_to_bf16_bits(np.asarray(a, np.float32))
    r = oracle.lm_head_stats(b([[1, 2], [-1, 0.5]]), b([[1, 0], [0.5, 0.5], [-1, 1]]), 1.0, want_logits=True)
    np.testing.assert_array_equal(r["logits"], [[1.0, 1.5, 1.0], [-1.0, -0.25, 1.5]])
    assert list(r["arg"]) == [1, 2] and list(r["max"]) == [1.5, 1.5] and list(r["gap"]) == [0.5, 1.75]
    np.testing.assert_allclose(r["sum"], [1 + 2 * np.exp(-0.5), 1 + np.exp(-2.5) + np.exp(-1.75)], rtol=1e-15)
    r2 = oracle.lm_head_stats(b([[1, 2], [-1, 0.5]]), b([[1, 0], [0.5, 0.5], [-1, 1]]), 0.5)
    np.testing.assert_allclose(r2["sum"], [1 + 2 * np.exp(-1.0), 1 + np.exp(-5.0) + np.exp(-3.5)], rtol=1e-15)


def test_scaling_and_permutation():
    h, w = synth.lm_head_inputs(4, 6, 96, 500)
    r = oracle.lm_head_stats(h, w, 1.0)
    h2 = h.copy()
    nz = h2 & 0x7FFF != 0
    h2[nz] += np.uint16(1 << 7)                      # exponent + 1: every hidden value doubled, exactly
    r2 = oracle.lm_head_stats(h2, w, 1.0)
    np.testing.assert_array_equal(r2["arg"], r["arg"])
    np.testing.assert_array_equal(r2["max"], 2 * r["max"])
    np.testing.assert_array_equal(r2["gap"], 2 * r["gap"])
    perm = np.random.default_rng(1).permutation(w.shape[0])
    r3 = oracle.lm_head_stats(h, np.ascontiguousarray(w[perm]), 1.0)
    np.testing.assert_array_equal(perm[r3["arg"]], r["arg"])
    np.testing.assert_array_equal(r3["max"], r["max"])
    np.testing.assert_allclose(r3["sum"], r["sum"], rtol=1e-13)
    np.testing.assert_array_equal(r3["gap"], r["gap"])


def test_agrees_with_row_statistics_of_its_own_logits():
    h, w = synth.lm_head_inputs(9, 7, 128, 3001)
    r = oracle.lm_head_stats(h, w, 1.3, want_logits=True)
    x32 = r["logits"].astype(np.float32)
    m, s, a = oracle.row_stats(x32, 1.3)
    exact = x32.astype(np.float64) == r["logits"]
    np.testing.assert_allclose(m, r["max"], rtol=1e-7)
    np.testing.assert_allclose(s, r["sum"], rtol=1e-5)
    for i in range(len(a)):                          # rounding to float can only merge near-equal values
        assert a[i] == r["arg"][i] or r["gap"][i] <= 1e-6 * abs(r["max"][i])
    assert exact.any()
