"""Pins for the head oracle: closed forms, invariants, a library restatement, brute force.

The paper fixes only that the head is MLP-based, conditioned on t and on the AR feature z,
and sampled in a few steps from shared noise; the AdaLN residual structure is this build's
reading. These tests pin the oracle's arithmetic to things that do not depend on itself.
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
import synth


def tiny_workload(**kw):
    base = dict(n=5, d=8, C=2, Dc=3, W=4, L=2, K=3, F=4)
    base.update(kw)
    return synth.workload("cfg1", **base)


def f64(bits):
    return synth.bf16_to_f32(bits).astype(np.float64)


def zero(w, *names):
    for k in names:
        w[k] = np.zeros_like(w[k])
    return w


def torch_head(w, cond_bits, noise, t_sched, idx):
    """fp64 restatement with torch library routines (linear, layer_norm, silu)."""
    W = {k: torch.from_numpy(f64(v)) for k, v in w.items()}
    Wd = W["Wc"].shape[0]
    L = W["Wmod"].shape[0]
    Fd = W["Wt1"].shape[1]
    z = torch.from_numpy(f64(cond_bits))[torch.from_numpy(idx).long()]
    x = torch.from_numpy(noise.astype(np.float64))[torch.from_numpy(idx).long()]
    c = F.linear(z, W["Wc"], W["bc"])
    t = torch.from_numpy(t_sched.astype(np.float64))
    half = Fd // 2
    freqs = torch.exp(-math.log(10000.0) * torch.arange(half, dtype=torch.float64) / half)
    for k in range(t.shape[0] - 1):
        arg = 1000.0 * t[k] * freqs
        e = torch.cat([torch.cos(arg), torch.sin(arg)])
        temb = F.linear(F.silu(F.linear(e, W["Wt1"], W["bt1"])), W["Wt2"], W["bt2"])
        s = F.silu(c + temb)
        h = F.linear(x, W["Win"], W["bin"])
        for b in range(L):
            sh, sc, g = F.linear(s, W["Wmod"][b], W["bmod"][b]).chunk(3, dim=-1)
            u = F.layer_norm(h, (Wd,), eps=1e-6) * (1 + sc) + sh
            h = h + g * F.linear(F.silu(F.linear(u, W["W1"][b], W["b1"][b])), W["W2"][b], W["b2"][b])
        sh, sc = F.linear(s, W["Wfm"], W["bfm"]).chunk(2, dim=-1)
        v = F.linear(F.layer_norm(h, (Wd,), eps=1e-6) * (1 + sc) + sh, W["Wout"], W["bout"])
        x = x + (t[k + 1] - t[k]) * v
    return x.numpy()


def inputs(wl, std=0.02):
    return (synth.head_weights(wl, std=std), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K))


def test_k0_returns_noise():
    wl = tiny_workload()
    w, cond, noise, _ = inputs(wl)
    idx = np.array([4, 0, 2], np.int32)
    out = oracle.head_sample(w, cond, noise, synth.t_sched(0), idx)
    assert np.array_equal(out[idx], noise[idx].astype(np.float64))
    assert np.all(out[[1, 3]] == 0.0)                       # rows of filtered tokens untouched


@pytest.mark.parametrize("K", [1, 4, 7])
def test_wout_zero_is_constant_velocity(K):
    """W_out = 0 makes v = b_out, so x^K = noise + (t_K - t_0) b_out for any K and schedule."""
    wl = synth.workload("cfg1", n=6, K=K)
    w, cond, noise, _ = inputs(wl, std=None)
    zero(w, "Wout")
    t = np.sort(np.random.default_rng(K).uniform(0.1, 0.9, size=K + 1)).astype(np.float32)
    idx = np.arange(6, dtype=np.int32)
    out = oracle.head_sample(w, cond, noise, t, idx)
    want = noise.astype(np.float64) + (float(t[-1]) - float(t[0])) * f64(w["bout"])[None, :]
    assert np.allclose(out, want, rtol=0, atol=1e-13)


def test_no_modulation_reduces_to_plain_ln_mlp_by_hand():
    """All modulation weights zero: blocks are the identity (gate = 0) and the final layer is
    v = W_out LN(W_in x + b_in) + b_out; checked with hand-written numpy at W = 4."""
    wl = tiny_workload(K=1)
    w, cond, noise, t = inputs(wl, std=None)
    zero(w, "Wmod", "bmod", "Wfm", "bfm")
    idx = np.arange(wl.n, dtype=np.int32)
    out = oracle.head_sample(w, cond, noise, t, idx)
    Win, b_in, Wout, bout = f64(w["Win"]), f64(w["bin"]), f64(w["Wout"]), f64(w["bout"])
    for j in range(wl.n):
        x = noise[j].astype(np.float64)
        h = Win @ x + b_in
        mu = h.sum() / 4.0
        var = ((h - mu) ** 2).sum() / 4.0
        u = (h - mu) / math.sqrt(var + 1e-6)
        v = Wout @ u + bout
        assert np.allclose(out[j], x + 1.0 * v, rtol=0, atol=1e-13)


def test_zero_gate_makes_blocks_identity_whatever_w1_w2():
    wl = tiny_workload()
    w, cond, noise, t = inputs(wl, std=None)
    Wd = wl.W
    w["Wmod"] = w["Wmod"].copy(); w["bmod"] = w["bmod"].copy()
    w["Wmod"][:, 2 * Wd:, :] = 0
    w["bmod"][:, 2 * Wd:] = 0
    idx = np.arange(wl.n, dtype=np.int32)
    a = oracle.head_sample(w, cond, noise, t, idx)
    w2 = dict(w)
    w2["W1"] = synth.f32_to_bf16(synth.bf16_to_f32(w["W1"]) * 3.0 + 1.0)
    w2["b2"] = synth.f32_to_bf16(synth.bf16_to_f32(w["b2"]) - 2.0)
    b = oracle.head_sample(w2, cond, noise, t, idx)
    assert np.array_equal(a, b)


def test_token_independence_and_idx_order():
    wl = synth.workload("cfg1", n=16)
    w, cond, noise, t = inputs(wl)
    idx = np.arange(16, dtype=np.int32)
    full = oracle.head_sample(w, cond, noise, t, idx)
    for j in (0, 7, 15):
        one = oracle.head_sample(w, cond, noise, t, np.array([j], np.int32))
        assert np.array_equal(one[j], full[j])                 # bit-identical
        assert np.all(np.delete(one, j, axis=0) == 0.0)
    perm = np.random.default_rng(0).permutation(16).astype(np.int32)
    assert np.array_equal(oracle.head_sample(w, cond, noise, t, perm), full)


def test_zero_length_step_changes_nothing():
    wl = synth.workload("cfg1", n=4, K=2)
    w, cond, noise, _ = inputs(wl, std=None)
    idx = np.arange(4, dtype=np.int32)
    a = oracle.head_sample(w, cond, noise, np.array([0.0, 0.5, 1.0], np.float32), idx)
    b = oracle.head_sample(w, cond, noise, np.array([0.0, 0.0, 0.5, 0.5, 1.0], np.float32), idx)
    assert np.allclose(a, b, rtol=0, atol=1e-14)


def test_time_direction_reversal_uses_signed_dt():
    """A one-step schedule (t0, t1) and its reverse use dt of opposite sign (same t_k = t0 would
    be needed for equality, so check only through W_out = 0: x moves by +-(t1 - t0) b_out)."""
    wl = synth.workload("cfg1", n=2, K=1)
    w, cond, noise, _ = inputs(wl, std=None)
    zero(w, "Wout")
    idx = np.arange(2, dtype=np.int32)
    fwd = oracle.head_sample(w, cond, noise, np.array([0.25, 1.0], np.float32), idx)
    bwd = oracle.head_sample(w, cond, noise, np.array([1.0, 0.25], np.float32), idx)
    assert np.allclose(fwd - noise, -(bwd - noise), rtol=0, atol=1e-14)
    assert np.allclose(fwd - noise, 0.75 * f64(w["bout"])[None, :], rtol=0, atol=1e-14)


@pytest.mark.parametrize("std", [0.02, None])
def test_matches_torch_fp64_restatement_cfg1(std):
    wl = synth.workload("cfg1")
    w, cond, noise, t = inputs(wl, std=std)
    idx = np.arange(0, wl.n, 3, dtype=np.int32)
    got = oracle.head_sample(w, cond, noise, t, idx)[idx]
    want = torch_head(w, cond, noise, t, idx)
    assert np.allclose(got, want, rtol=1e-11, atol=1e-12)


def test_matches_torch_fp64_restatement_odd_shapes():
    wl = synth.workload("cfg1", n=7, C=5, Dc=9, W=12, L=3, K=5, F=6)
    w, cond, noise, _ = inputs(wl, std=None)
    t = np.array([0.0, 0.1, 0.15, 0.4, 0.8, 1.0], np.float32)
    idx = np.array([6, 1, 3], np.int32)
    got = oracle.head_sample(w, cond, noise, t, idx)[idx]
    want = torch_head(w, cond, noise, t, idx)
    assert np.allclose(got, want, rtol=1e-11, atol=1e-12)


def test_brute_force_python_loops_tiny():
    """Per-token scalar Python, column-major accumulation order, on a tiny head."""
    wl = tiny_workload(n=3, K=2)
    w, cond, noise, t = inputs(wl, std=None)
    P = {k: f64(v) for k, v in w.items()}
    C, Dc, Wd, L, Fd = wl.C, wl.Dc, wl.W, wl.L, wl.F
    silu = lambda a: a / (1.0 + math.exp(-a))

    def lin(Wm, b, x):
        y = [float(b[o]) for o in range(len(b))]
        for i in range(len(x)):                      # input-major loop order, unlike the oracle
            for o in range(len(b)):
                y[o] += float(Wm[o][i]) * x[i]
        return y

    def ln(h):
        mu = sum(h) / len(h)
        var = sum((v - mu) ** 2 for v in h) / len(h)
        return [(v - mu) / math.sqrt(var + 1e-6) for v in h]

    idx = np.arange(3, dtype=np.int32)
    got = oracle.head_sample(w, cond, noise, t, idx)
    zc = f64(cond)
    for j in range(3):
        x = [float(v) for v in noise[j]]
        c = lin(P["Wc"], P["bc"], [float(v) for v in zc[j]])
        for k in range(2):
            tk = float(t[k])
            half = Fd // 2
            e = [math.cos(1000.0 * tk * 10000.0 ** (-f / half)) for f in range(half)] + \
                [math.sin(1000.0 * tk * 10000.0 ** (-f / half)) for f in range(half)]
            temb = lin(P["Wt2"], P["bt2"], [silu(v) for v in lin(P["Wt1"], P["bt1"], e)])
            s = [silu(c[i] + temb[i]) for i in range(Wd)]
            h = lin(P["Win"], P["bin"], x)
            for b in range(L):
                mod = lin(P["Wmod"][b], P["bmod"][b], s)
                n_ = ln(h)
                u = [n_[i] * (1.0 + mod[Wd + i]) + mod[i] for i in range(Wd)]
                r = lin(P["W2"][b], P["b2"][b], [silu(v) for v in lin(P["W1"][b], P["b1"][b], u)])
                h = [h[i] + mod[2 * Wd + i] * r[i] for i in range(Wd)]
            mod = lin(P["Wfm"], P["bfm"], s)
            n_ = ln(h)
            u = [n_[i] * (1.0 + mod[Wd + i]) + mod[i] for i in range(Wd)]
            v = lin(P["Wout"], P["bout"], u)
            dt = float(t[k + 1]) - float(t[k])
            x = [x[i] + dt * v[i] for i in range(C)]
        assert np.allclose(got[j], x, rtol=1e-12, atol=1e-13)


def test_time_embedding_closed_forms():
    wl = synth.workload("cfg1", F=8)
    w = synth.head_weights(wl, std=None)
    P = {k: f64(v) for k, v in w.items()}
    silu = lambda a: a / (1.0 + np.exp(-a))
    # t = 0: e = [1,1,1,1, 0,0,0,0]
    e0 = np.array([1.0] * 4 + [0.0] * 4)
    want0 = P["Wt2"] @ silu(P["Wt1"] @ e0 + P["bt1"]) + P["bt2"]
    assert np.allclose(oracle.time_embedding(w, 0.0), want0, rtol=1e-12, atol=1e-13)
    # general t: frequencies 10000^(-f/4) = 1, 0.1, 0.01, 0.001 ; argument 1000 t w_f
    t = np.float32(0.3125)
    arg = 1000.0 * float(t) * np.array([1.0, 0.1, 0.01, 0.001])
    e = np.concatenate([np.cos(arg), np.sin(arg)])
    want = P["Wt2"] @ silu(P["Wt1"] @ e + P["bt1"]) + P["bt2"]
    assert np.allclose(oracle.time_embedding(w, float(t)), want, rtol=1e-11, atol=1e-12)


def test_layer_norm_against_torch_and_moments():
    rng = np.random.default_rng(5)
    h = rng.normal(size=257) * 3.0 + 10.0
    got = oracle.layer_norm(h)
    want = F.layer_norm(torch.from_numpy(h), (257,), eps=1e-6).numpy()
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    assert abs(got.mean()) < 1e-13
    assert abs((got ** 2).mean() - h.var() / (h.var() + 1e-6)) < 1e-12
    # constant row: variance 0, eps keeps it finite: output exactly 0
    assert np.all(oracle.layer_norm(np.full(16, 2.5)) == 0.0)


def test_golden_cfg1_fixture():
    """The stored cfg1 values were written by tests/golden/make_golden.py, which calls only the
    oracle; this guards the oracle against silent arithmetic changes."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "oracle_cfg1.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    wl = synth.workload("cfg1")
    f = synth.features(wl)
    H = oracle.entropy(f)
    w, cond, noise, t = inputs(wl)
    toks = sorted({int(r[1]) for r in rows if r[0] == "out"})
    out = oracle.head_sample(w, cond, noise, t, np.array(toks, np.int32))
    for r in rows:
        if r[0] == "H":
            assert abs(H[int(r[1])] - float.fromhex(r[2])) <= 1e-13 * max(1.0, abs(H[int(r[1])]))
        elif r[0] == "out":
            assert abs(out[int(r[1]), int(r[2])] - float.fromhex(r[3])) <= 1e-12
