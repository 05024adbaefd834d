"""Pins for the gate oracle: closed forms, invariants, library special cases, brute force.

The paper prints no worked numeric example of an entropy value, so the oracle is pinned to
what the definition (entropy of the softmax-normalised row, natural log, H = -L_entropy;
Algorithm 1 drops a token iff H < tau) and the mathematics fix.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import synth

LN = math.log


def bits(x):
    """float array -> bf16 bits; asserts the values are exactly representable."""
    x = np.asarray(x, dtype=np.float32)
    b = synth.f32_to_bf16(x)
    back = synth.bf16_to_f32(b)
    assert np.array_equal(back, x) or np.array_equal(np.isnan(back), np.isnan(x)), "not bf16-exact"
    return b


@pytest.mark.parametrize("d", [1, 2, 8, 256, 768, 5120])
@pytest.mark.parametrize("v", [0.0, -3.5, 12.0])
def test_uniform_row_is_ln_d(d, v):
    H = oracle.entropy(bits(np.full((3, d), v)))
    assert np.allclose(H, LN(d), rtol=0, atol=1e-12)


def test_one_hot_limit_is_zero():
    for d in (8, 256, 5120):
        x = np.zeros((1, d), np.float32)
        x[0, d // 3] = 100.0
        H = oracle.entropy(bits(x))
        # leading term of the two-level closed form for alpha >> 1: (d-1) e^-alpha (alpha + 1);
        # the "+1" part (from the dominant channel's own -p ln p, p = 1 - 1e-41) is below fp64
        # resolution of 1, so only 1 % agreement is asked at this magnitude (1e-38 absolute)
        lead = (d - 1) * math.exp(-100.0) * 101.0
        assert 0.0 <= H[0] < 1e-35 and abs(H[0] - lead) < 0.011 * lead


@pytest.mark.parametrize("d,a,alpha", [(8, 1, 1.5), (256, 7, 3.0), (768, 100, -2.0), (1024, 1, 8.0),
                                       (5120, 5119, 0.5)])
def test_two_level_row_closed_form(d, a, alpha):
    """a channels at alpha, d-a at 0: S = a e^alpha + d - a, H = ln S - a alpha e^alpha / S."""
    x = np.zeros((1, d), np.float32)
    pos = np.random.default_rng(d).permutation(d)[:a]
    x[0, pos] = alpha
    S = a * math.exp(alpha) + d - a
    want = LN(S) - a * alpha * math.exp(alpha) / S
    H = oracle.entropy(bits(x))
    assert abs(H[0] - want) < 1e-12 * max(1.0, abs(want))


def test_three_level_row_closed_form():
    """-sum p ln p written out for probabilities known in closed form (1/2, 1/4, 1/8, 1/8)."""
    ln2 = LN(2.0)
    # logits ln(p) up to a shift: use exact powers of two -> x = log2(p) * ln2 is not bf16-exact,
    # so build the row from repeated channels instead: counts 4,2,1,1 of equal logits.
    x = np.zeros((1, 8), np.float32)          # 8 equal channels: p = 1/8 each, H = ln 8
    assert abs(oracle.entropy(bits(x))[0] - 3 * ln2) < 1e-14
    # groups: merge channels by giving them -inf except one representative carrying ln(count)
    # is not representable; instead check the grouping identity H(parts) = H(groups) + sum_g P_g H(within g)
    rng = np.random.default_rng(0)
    row = np.round(rng.normal(size=16) * 4) / 4   # multiples of 0.25: bf16-exact
    H_all = oracle.entropy(bits(row[None, :]))[0]
    p = np.exp(row - row.max()); p /= p.sum()
    Pg = np.array([p[:5].sum(), p[5:].sum()])
    Hg = -(Pg * np.log(Pg)).sum()
    Hin = [oracle.entropy(bits(row[None, :5]))[0], oracle.entropy(bits(row[None, 5:]))[0]]
    assert abs(H_all - (Hg + Pg[0] * Hin[0] + Pg[1] * Hin[1])) < 1e-12


def test_invariants_permutation_shift_duplication():
    rng = np.random.default_rng(1)
    x = np.round(rng.normal(size=(5, 96)) * 8) / 8            # multiples of 1/8, |x| small: bf16-exact
    H = oracle.entropy(bits(x))
    perm = rng.permutation(96)
    assert np.allclose(oracle.entropy(bits(x[:, perm])), H, rtol=0, atol=1e-13)
    assert np.allclose(oracle.entropy(bits(x + 4.0)), H, rtol=0, atol=1e-13)
    assert np.allclose(oracle.entropy(bits(np.concatenate([x, x], axis=1))), H + LN(2.0), rtol=0, atol=1e-13)
    # scaling the logits is NOT an invariance (guards against a stray temperature)
    assert not np.allclose(oracle.entropy(bits(x * 2.0)), H, atol=1e-3)


def test_matches_torch_and_scipy_fp64():
    import scipy.special
    wl = synth.workload("cfg1")
    f = synth.features(wl)
    x = synth.bf16_to_f32(f).astype(np.float64)
    H = oracle.entropy(f)
    Ht = torch.distributions.Categorical(logits=torch.from_numpy(x)).entropy().numpy()
    assert np.allclose(H, Ht, rtol=1e-12, atol=1e-13)
    Hs = scipy.special.entr(scipy.special.softmax(x, axis=1)).sum(axis=1)
    assert np.allclose(H, Hs, rtol=1e-12, atol=1e-13)
    # heavy-tailed rows too
    wl4 = synth.workload("cfg4")
    f4 = synth.features(wl4, 100, 64)
    x4 = synth.bf16_to_f32(f4).astype(np.float64)
    Ht4 = torch.distributions.Categorical(logits=torch.from_numpy(x4)).entropy().numpy()
    assert np.allclose(oracle.entropy(f4), Ht4, rtol=1e-11, atol=1e-13)


def test_brute_force_two_forms_tiny():
    """Pure-Python literal -sum p ln p, and the ln S - T/S rearrangement, on tiny rows."""
    rng = np.random.default_rng(2)
    x = np.round(rng.normal(size=(6, 11)) * 16) / 16
    H = oracle.entropy(bits(x))
    for i in range(x.shape[0]):
        row = [float(v) for v in x[i]]
        m = max(row)
        S = sum(math.exp(v - m) for v in row)
        lit = -sum((math.exp(v - m) / S) * math.log(math.exp(v - m) / S) for v in row)
        T = sum((v - m) * math.exp(v - m) for v in row)
        alt = math.log(S) - T / S
        assert abs(H[i] - lit) < 1e-13 and abs(H[i] - alt) < 1e-13


def test_minus_inf_channels_contribute_nothing_and_bad_rows_are_dropped():
    rng = np.random.default_rng(3)
    x = np.round(rng.normal(size=(1, 24)) * 4) / 4
    xi = np.concatenate([x, np.full((1, 8), -np.inf)], axis=1).astype(np.float32)
    fb = synth.f32_to_bf16(xi)
    assert abs(oracle.entropy(fb)[0] - oracle.entropy(bits(x))[0]) < 1e-14
    bad = np.zeros((3, 8), np.float32)
    bad[0, :] = -np.inf
    bad[1, 2] = np.nan
    bad[2, 5] = np.inf
    H, mask, idx, count = oracle.gate(synth.f32_to_bf16(bad), -1.0)
    assert np.all(np.isnan(H)) and count == 0 and mask.sum() == 0


def test_threshold_direction_and_tie():
    """Drop iff H < tau (Algorithm 1); equality keeps. tau is a float32 widened to double."""
    d = 256
    f = bits(np.zeros((1, d)))
    H = oracle.entropy(f)[0]
    t32 = np.float32(H)
    lo, hi = np.nextafter(t32, np.float32(-np.inf)), np.nextafter(t32, np.float32(np.inf))
    assert oracle.gate(f, lo)[3] == 1
    assert oracle.gate(f, hi)[3] == 0
    assert oracle.gate(f, t32)[3] == (1 if H >= float(t32) else 0)
    # an exact tie: d = 1 gives H = 0 exactly; tau = 0 keeps, tau = tiny positive drops
    f1 = bits(np.zeros((4, 1)))
    assert oracle.gate(f1, 0.0)[3] == 4
    assert oracle.gate(f1, 1e-30)[3] == 0


def test_compaction_is_ascending_positions_of_mask():
    wl = synth.workload("cfg2", n=4099)
    f = synth.features(wl)
    H = oracle.entropy(f)
    for q in (0.0, 0.3, 0.9, 1.0):
        tau = float(np.quantile(H, q)) if q > 0 else -1.0
        Hg, mask, idx, count = oracle.gate(f, tau)
        assert np.array_equal(Hg, H)
        want_mask = (H >= float(np.float32(tau))).astype(np.uint8)
        assert np.array_equal(mask, want_mask)
        assert count == int(want_mask.sum()) == idx.shape[0]
        assert np.array_equal(idx, np.flatnonzero(want_mask).astype(np.int32))
    # empty input
    H0, m0, i0, c0 = oracle.gate(np.zeros((0, 8), np.uint16), 0.0)
    assert c0 == 0 and m0.shape == (0,)


def test_entropy_bounds_on_workload_rows():
    for name, rows in (("cfg1", 64), ("cfg2", 512), ("cfg3", 256), ("cfg4", 64)):
        wl = synth.workload(name)
        H = oracle.entropy(synth.features(wl, 0, rows))
        assert np.all(H >= 0.0) and np.all(H <= LN(wl.d) + 1e-12)
