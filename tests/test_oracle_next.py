"""Pins for the oracle's later-stage functions: block-prefix early stop (Algorithm 1, Step 1), the
threshold equation tau = 0.3 mean - 0.1 std, the accepted-prefix length (Algorithm 1, Step 4) and the
generalised linear sampler step. Each is checked against closed forms, special cases that reduce to an
already pinned function or a library routine, and brute force written differently from the oracle."""
import numpy as np
import pytest

import oracle
import synth


def rows_with_entropy_levels(levels, d=64):
    """bf16 rows whose entropies are known in closed form: level a in 1..d -> a equal large channels,
    the rest far below: H = ln a (to ~1e-12 with a 60-unit gap)."""
    out = np.empty((len(levels), d), dtype=np.uint16)
    for i, a in enumerate(levels):
        x = np.full(d, -60.0, np.float32)
        x[:a] = 0.0
        out[i] = synth.f32_to_bf16(x)
    return out


def test_gamma_one_reduces_to_the_per_token_gate():
    wl = synth.workload("cfg1", n=200)
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    tau = float(np.median(H))
    _, mask, idx, count = oracle.gate(bits, tau)
    Hs, mask_b, idx_b, count_b, ln = oracle.gate_blocks(bits, 1, 1, tau)
    assert np.array_equal(Hs, H) and np.array_equal(mask_b, mask) and np.array_equal(idx_b, idx)
    assert count_b == count and np.array_equal(ln, mask.astype(np.int32))


@pytest.mark.parametrize("gamma", [2, 3, 8, 64, 1000])
def test_block_prefix_brute_force_and_closed_form_levels(gamma):
    rng = np.random.default_rng(gamma)
    levels = rng.integers(1, 33, size=157)
    bits = rows_with_entropy_levels(levels)
    tau = float(np.log(7.5))                         # keep iff level >= 8
    Hs, mask, idx, count, ln = oracle.gate_blocks(bits, 1, gamma, tau)
    assert np.allclose(Hs, np.log(levels), atol=1e-9)
    want = np.zeros(len(levels), np.uint8)
    want_len = []
    for b0 in range(0, len(levels), gamma):
        blk = levels[b0:b0 + gamma]
        bad = np.flatnonzero(blk < 8)
        keep = len(blk) if len(bad) == 0 else int(bad[0])
        want[b0:b0 + keep] = 1
        want_len.append(keep)
    assert np.array_equal(mask, want)
    assert np.array_equal(ln, np.array(want_len, np.int32))
    assert count == int(want.sum()) and np.array_equal(idx, np.flatnonzero(want).astype(np.int32))


def test_rows_per_token_takes_the_mean_of_row_entropies():
    levels = np.array([1, 4, 16, 64, 2, 2, 8, 32, 64, 64, 64, 64], dtype=np.int64)   # 3 tokens x 4 rows
    bits = rows_with_entropy_levels(levels)
    Hs, mask, idx, count, ln = oracle.gate_blocks(bits, 4, 3, tau=float(np.log(5.0)))
    assert np.allclose(Hs, np.log(levels).reshape(3, 4).mean(axis=1), atol=1e-9)
    # token means: ln(4096)/4 = ln 8 ; ln(1024)/4 ~ ln 5.66 ; ln 64  -> all >= ln 5: whole block kept
    assert mask.tolist() == [1, 1, 1] and ln.tolist() == [3] and count == 3
    _, mask2, _, _, ln2 = oracle.gate_blocks(bits, 4, 3, tau=float(np.log(6.0)))
    assert mask2.tolist() == [1, 0, 0] and ln2.tolist() == [1]      # token 1 falls below: it and token 2 go


def test_nan_row_ends_the_block():
    bits = rows_with_entropy_levels([32, 32, 32, 32])
    bits[2, 5] = 0x7FC0                                               # NaN
    _, mask, _, _, ln = oracle.gate_blocks(bits, 1, 4, tau=0.0)
    assert mask.tolist() == [1, 1, 0, 0] and ln.tolist() == [2]


def test_tau_calibration_against_numpy_and_closed_forms():
    rng = np.random.default_rng(3)
    H = rng.uniform(0.5, 6.0, size=1001)
    m, s, t = oracle.tau_calibrate(H)
    assert abs(m - np.mean(H)) < 1e-12 and abs(s - np.std(H)) < 1e-12
    assert abs(t - (0.3 * np.mean(H) - 0.1 * np.std(H))) < 1e-12
    m, s, t = oracle.tau_calibrate(np.full(17, 2.5))
    assert (m, s) == (2.5, 0.0) and abs(t - 0.75) < 1e-15
    m, s, t = oracle.tau_calibrate(np.array([1.0, 3.0] * 50))        # two-point: mean 2, std 1
    assert abs(m - 2.0) < 1e-15 and abs(s - 1.0) < 1e-15 and abs(t - 0.5) < 1e-15


@pytest.mark.parametrize("gamma", [1, 4, 8, 37])
def test_accept_prefix_brute_force(gamma):
    rng = np.random.default_rng(gamma)
    n = 203
    r = rng.uniform(0, 1, n).astype(np.float32)
    ratio = rng.uniform(0.3, 1.5, n).astype(np.float32)
    got = oracle.accept_prefix(r, ratio, gamma)
    want = []
    for b0 in range(0, n, gamma):
        rej = [i for i in range(b0, min(n, b0 + gamma)) if r[i] > ratio[i]]
        want.append((rej[0] - b0) if rej else min(n, b0 + gamma) - b0)
    assert got.tolist() == want
    assert oracle.accept_prefix(np.zeros(9, np.float32), np.ones(9, np.float32), 4).tolist() == [4, 4, 1]
    assert oracle.accept_prefix(np.ones(8, np.float32), np.zeros(8, np.float32), 4).tolist() == [0, 0]
    eq = np.full(4, 0.5, np.float32)                                  # r == ratio is not a rejection (strict >)
    assert oracle.accept_prefix(eq, eq, 4).tolist() == [4]


@pytest.mark.parametrize("gamma", [1, 5, 8])
def test_accept_prefix_after_early_stop_brute_force(gamma):
    """Algorithm 1 runs Step 4 on the draft that Step 1 left: len(draft_tokens) is the truncated length, so a
    rejection at or beyond it is never seen and the accepted count is capped by it."""
    rng = np.random.default_rng(100 + gamma)
    n = 131
    nb = (n + gamma - 1) // gamma
    r = rng.uniform(0, 1, n).astype(np.float32)
    ratio = rng.uniform(0.2, 1.4, n).astype(np.float32)
    full = np.array([min(gamma, n - b * gamma) for b in range(nb)], np.int32)
    kept = np.minimum(rng.integers(0, gamma + 1, nb).astype(np.int32), full)
    got = oracle.accept_prefix(r, ratio, gamma, kept)
    want = []
    for b in range(nb):
        draft = range(b * gamma, b * gamma + int(kept[b]))
        rej = [i - b * gamma for i in draft if r[i] > ratio[i]]
        want.append(min(rej + [int(kept[b])]))
    assert got.tolist() == want
    assert np.all(got <= kept)
    # no truncation recorded = the untruncated call; an all-rejecting block of kept length 0 accepts nothing
    assert oracle.accept_prefix(r, ratio, gamma, full).tolist() == oracle.accept_prefix(r, ratio, gamma).tolist()
    assert oracle.accept_prefix(np.zeros(8, np.float32), np.ones(8, np.float32), 4, np.array([0, 3])).tolist() == [0, 3]


def test_early_stop_then_accept_prefix_compose():
    """Step 1 -> Step 4 as the algorithm writes them: the kept lengths of the block-prefix gate feed the
    accepted-prefix count; with ratios that never reject, the accepted length is exactly the kept length."""
    wl = synth.workload("cfg2", n=96)
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    tau = float(np.quantile(H, 0.25))
    _, _, _, _, ln = oracle.gate_blocks(bits, 1, 8, tau)
    r = np.full(96, 0.5, np.float32)
    assert oracle.accept_prefix(r, np.ones(96, np.float32), 8, ln).tolist() == ln.tolist()
    assert 0 < ln.sum() < 96


def test_linear_sampler_with_euler_coefficients_is_the_euler_sampler():
    wl = synth.workload("cfg1", n=40, K=5)
    w, cond, noise = synth.head_weights(wl, std=None), synth.cond(wl), synth.noise(wl)
    t = np.sort(np.random.default_rng(0).uniform(0, 1, 6)).astype(np.float32)
    idx = np.arange(40, dtype=np.int32)
    coef = np.stack([np.ones(5), (t[1:].astype(np.float64) - t[:-1].astype(np.float64)), np.zeros(5)], axis=1)
    a = oracle.head_sample(w, cond, noise, t, idx)
    b = oracle.head_sample_coef(w, cond, noise, t[:-1], coef.astype(np.float32), idx)
    assert np.abs(a - b).max() <= 1e-7 * np.abs(a).max()              # coefficients pass through float32


def test_linear_sampler_closed_form_when_the_head_output_is_constant():
    """W_out = 0 makes v = b_out for every token and step, so the K-step recurrence has the closed form
    x_K = (prod ax) x_0 + sum_k (prod_{j>k} ax_j) (av_k b_out + an_k z_k)."""
    wl = synth.workload("cfg1", n=12, K=4)
    w = synth.head_weights(wl)
    w["Wout"] = np.zeros_like(w["Wout"])
    cond, noise = synth.cond(wl), synth.noise(wl)
    rng = np.random.default_rng(5)
    coef = rng.uniform(-1.2, 1.2, size=(4, 3)).astype(np.float32)
    z = rng.standard_normal((4, 12, wl.C)).astype(np.float32)
    t_in = np.array([0.9, 0.6, 0.3, 0.1], np.float32)
    got = oracle.head_sample_coef(w, cond, noise, t_in, coef, np.arange(12, dtype=np.int32), step_noise=z)
    bout = synth.bf16_to_f32(w["bout"]).astype(np.float64)
    c = coef.astype(np.float64)
    want = np.prod(c[:, 0]) * noise.astype(np.float64)
    for k in range(4):
        tail = np.prod(c[k + 1:, 0])
        want += tail * (c[k, 1] * bout[None, :] + c[k, 2] * z[k].astype(np.float64))
    assert np.abs(got - want).max() < 1e-12


def test_ddim_coefficients_reproduce_a_textbook_ddim_step_by_hand():
    """eps-prediction step x' = sqrt(ab') x0 + sqrt(1 - ab') eps with x0 = (x - sqrt(1 - ab) eps) / sqrt(ab),
    written out on a W_out = 0 head (eps = b_out) and compared with the (ax, av) form the sampler takes."""
    wl = synth.workload("cfg1", n=6, K=1)
    w = synth.head_weights(wl)
    w["Wout"] = np.zeros_like(w["Wout"])
    cond, noise = synth.cond(wl), synth.noise(wl)
    ab, abn = 0.35, 0.8
    ax = np.sqrt(abn / ab)
    av = np.sqrt(1 - abn) - ax * np.sqrt(1 - ab)
    coef = np.array([[ax, av, 0.0]], np.float32)
    got = oracle.head_sample_coef(w, cond, noise, np.array([0.5], np.float32), coef, np.arange(6, dtype=np.int32))
    eps = synth.bf16_to_f32(w["bout"]).astype(np.float64)[None, :]
    x = noise.astype(np.float64)
    x0 = (x - np.sqrt(1 - ab) * eps) / np.sqrt(ab)
    want = np.sqrt(abn) * x0 + np.sqrt(1 - abn) * eps
    assert np.abs(got - want).max() < 1e-6                           # float32 coefficients
