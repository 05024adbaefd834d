"""The rounding model (rounding_model.py) is pinned to the oracle, and it derives what the parity bar of the
head can and cannot promise: with bf16 operands the error floor grows with depth and with the step size, and
at the deepest single-step workload (cfg 3 at K = 1) a small tail of tokens reaches the 2e-2 x RMS bar by
rounding alone. CPU only."""
import numpy as np
import pytest

import oracle
import rounding_model as rm
import synth


def test_without_rounding_the_model_is_the_oracle():
    wl = synth.workload("cfg1", n=40)
    w, cond, noise, t = synth.head_weights(wl, std=None), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K)
    toks = np.array([3, 0, 17, 39, 8], np.int32)
    want = oracle.head_sample(w, cond, noise, t, toks)[toks]
    got = rm.head(w, cond, noise, t, toks, rounded=())
    assert np.abs(got - want).max() <= 1e-11 * np.abs(want).max()


def test_each_rounding_point_moves_the_result_by_about_one_bf16_ulp_not_more():
    """A rounding inserted at the wrong place or applied twice would show as an error far above 2^-9."""
    wl = synth.workload("cfg1", n=64, K=1)
    w, cond, noise, t = synth.head_weights(wl, std=None), synth.cond(wl), synth.noise(wl), synth.t_sched(1)
    toks = np.arange(64)
    ref = rm.head(w, cond, noise, t, toks, rounded=())
    for p in rm.POINTS:
        r = rm.error_ratio(rm.head(w, cond, noise, t, toks, rounded=(p,)), ref)
        assert 1e-5 < np.median(r) < 8e-3, (p, np.median(r))


@pytest.mark.parametrize("K,lo,hi", [(1, 5.0e-3, 8.5e-3), (4, 2.5e-3, 5.0e-3)])
def test_error_floor_of_bf16_operands_on_the_deep_head(K, lo, hi):
    """cfg 3 shape (W = 1536, 6 blocks): rounding alone puts the median token at about a third of the bar at
    K = 1 and a fifth at K = 4 (four quarter steps average), and the one-step tail comes close to the bar."""
    wl = synth.workload("cfg3", K=K)
    w, t = synth.head_weights(wl), synth.t_sched(K)
    toks = np.sort(np.random.default_rng(K).choice(wl.n, 192, replace=False))
    cond = np.zeros((wl.n, wl.Dc), np.uint16)
    noise = np.zeros((wl.n, wl.C), np.float32)
    for tk in toks:
        cond[tk], noise[tk] = synth.cond(wl, int(tk), 1)[0], synth.noise(wl, int(tk), 1)[0]
    ref = rm.head(w, cond, noise, t, toks, rounded=())
    r = rm.error_ratio(rm.head(w, cond, noise, t, toks), ref)
    assert lo < np.median(r) < hi, np.median(r)
    if K == 1:
        assert np.quantile(r, 0.99) > 1.0e-2          # the tail is real: 1 % of the tokens use half of the bar
