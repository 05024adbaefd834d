"""GPU parity of the K-step head against the fp64 oracle, through the C ABI.

Agreement bar: per token, max |out - oracle| <= 2e-2 * RMS(oracle row) (bf16 GEMM operands, fp32
accumulation on the GPU; no rounding in the oracle). The same bar is applied to the velocity
(out - noise) on one-step runs, where the noise no longer props up the RMS. On the full-size
workloads, where several hundred tokens are compared, a token that misses the bar is looked up in
the CPU rounding model (gpu_util.assert_head_parity): it may pass only if bf16 rounding alone
already puts it there.
"""
import numpy as np
import pytest
import torch

import oracle
import rounding_model
import synth
import paper_2512_08537_b200 as ardiff
from gpu_util import assert_head_parity, dev_bf16, dev_f32, require_cuda

pytestmark = pytest.mark.gpu

REL_TOL = 2e-2
SENTINEL = -777.0


def make_head(wl, weights, max_tokens=None, K_max=None):
    return ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K if K_max is None else K_max,
                       wl.n if max_tokens is None else max_tokens, weights)


def run_head(head, cond_bits, noise, t, idx_np, n_rows=None):
    dev = require_cuda()
    cond = dev_bf16(cond_bits)
    nz = dev_f32(noise)
    idx = torch.from_numpy(np.ascontiguousarray(idx_np, dtype=np.int32)).to(dev)
    if idx.numel() == 0:
        idx = torch.zeros(1, dtype=torch.int32, device=dev)
    count = torch.tensor([len(idx_np)], dtype=torch.int32, device=dev)
    out = torch.full(noise.shape, SENTINEL, dtype=torch.float32, device=dev)
    head.ardiff_head_sample(cond, nz, t, idx, count, out)
    st = head.status()
    assert st == 0, ardiff.strerror(st)
    return out.cpu().numpy()


def assert_parity(got, want, rows, what="out"):
    err = np.abs(got[rows].astype(np.float64) - want[rows]).max(axis=1)
    rms = np.sqrt((want[rows] ** 2).mean(axis=1))
    worst = float((err / rms).max())
    assert worst <= REL_TOL, f"{what}: worst max|err|/rms = {worst:.3e}"
    return worst


def sample_tokens(idx, extra=96, seed=0):
    """First tile, a middle tile, the last (ragged) tile, and some random survivors."""
    S = len(idx)
    pos = set(range(min(S, 128)))
    pos |= set(range(max(0, (S // 256) * 128), min(S, (S // 256) * 128 + 64)))
    pos |= set(range(max(0, S - (S % 128 or 128)), S))
    rng = np.random.default_rng(seed)
    pos |= set(int(p) for p in rng.integers(0, S, size=extra))
    return np.array(sorted(pos), dtype=np.int64)


def test_cfg1_all_tokens_gate_then_head():
    dev = require_cuda()
    wl = synth.workload("cfg1")
    feat_bits = synth.features(wl)
    H = oracle.entropy(feat_bits)
    tau = float(np.median(H))
    _, mask_o, idx_o, count_o = oracle.gate(feat_bits, tau)
    w, cond_bits, noise, t = synth.head_weights(wl), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K)
    want = oracle.head_sample(w, cond_bits, noise, t, idx_o)
    head = make_head(wl, w)
    mask, idx, count, _ = ardiff.ardiff_entropy_gate(dev_bf16(feat_bits), tau)
    out = torch.full(noise.shape, SENTINEL, dtype=torch.float32, device=dev)
    head.ardiff_head_sample(dev_bf16(cond_bits), dev_f32(noise), t, idx, count, out)
    assert head.status() == 0
    got = out.cpu().numpy()
    assert int(count.item()) == count_o
    assert_parity(got, want, idx_o)
    dropped = np.flatnonzero(mask_o == 0)
    assert np.all(got[dropped] == SENTINEL)          # rows of filtered tokens are never written
    head.close()


@pytest.mark.parametrize("std", [0.02, None])
@pytest.mark.parametrize("count", [1, 64, 127, 128, 129, 300])
def test_small_head_ragged_counts(std, count):
    wl = synth.workload("cfg1", n=320)
    w, cond_bits, noise, t = synth.head_weights(wl, std=std), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K)
    idx = np.random.default_rng(count).permutation(wl.n)[:count].astype(np.int32)   # any order
    want = oracle.head_sample(w, cond_bits, noise, t, idx)
    head = make_head(wl, w)
    got = run_head(head, cond_bits, noise, t, idx)
    assert_parity(got, want, idx)
    rest = np.setdiff1d(np.arange(wl.n), idx)
    assert np.all(got[rest] == SENTINEL)
    head.close()


@pytest.mark.parametrize("std", [0.02, None])
def test_velocity_parity_one_step(std):
    wl = synth.workload("cfg1", n=256, K=1)
    w, cond_bits, noise, t = synth.head_weights(wl, std=std), synth.cond(wl), synth.noise(wl), synth.t_sched(1)
    idx = np.arange(wl.n, dtype=np.int32)
    want = oracle.head_sample(w, cond_bits, noise, t, idx)
    head = make_head(wl, w)
    got = run_head(head, cond_bits, noise, t, idx)
    assert_parity(got - noise, want - noise, idx, "velocity")
    head.close()


def test_k0_copies_noise_and_count0_writes_nothing():
    wl = synth.workload("cfg1", n=200)
    w, cond_bits, noise = synth.head_weights(wl), synth.cond(wl), synth.noise(wl)
    head = make_head(wl, w)
    idx = np.arange(0, 200, 3, dtype=np.int32)
    got = run_head(head, cond_bits, noise, synth.t_sched(0), idx)
    assert np.array_equal(got[idx], noise[idx])
    assert np.all(got[np.setdiff1d(np.arange(200), idx)] == SENTINEL)
    got0 = run_head(head, cond_bits, noise, synth.t_sched(4), np.zeros(0, np.int32))
    assert np.all(got0 == SENTINEL)
    head.close()


def test_nonuniform_schedule_and_k_sweep():
    wl = synth.workload("cfg1", n=192, K=8)
    w, cond_bits, noise = synth.head_weights(wl, std=None), synth.cond(wl), synth.noise(wl)
    head = make_head(wl, w, K_max=8)
    idx = np.arange(wl.n, dtype=np.int32)
    for K in (1, 2, 3, 8):
        t = np.sort(np.random.default_rng(K).uniform(0.0, 1.0, size=K + 1)).astype(np.float32)
        want = oracle.head_sample(w, cond_bits, noise, t, idx)
        got = run_head(head, cond_bits, noise, t, idx)
        assert_parity(got, want, idx, f"K={K}")
    # reversed time direction
    t = np.array([1.0, 0.5, 0.0], np.float32)
    assert_parity(run_head(head, cond_bits, noise, t, idx), oracle.head_sample(w, cond_bits, noise, t, idx), idx)
    head.close()


def test_two_calls_on_one_head_give_identical_results():
    wl = synth.workload("cfg1", n=300)
    w, cond_bits, noise, t = synth.head_weights(wl), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K)
    head = make_head(wl, w)
    idx = np.arange(wl.n, dtype=np.int32)
    a = run_head(head, cond_bits, noise, t, idx)
    b = run_head(head, cond_bits, noise, t, idx)
    assert np.array_equal(a, b)
    head.close()


@pytest.mark.parametrize("name,runs,K", [("cfg2", 12, 4), ("cfg3", 4, 2)])
def test_full_size_runs_are_bit_identical(name, runs, K):
    """The kernel's arithmetic has a fixed order, so equal inputs must give equal bits however the
    items of the many CTAs interleave. A tile read before its producer's writes were visible (an
    ordering bug between CTAs) shows up here as a run that differs; the cache flush and the
    varying survivor counts in between change the timing from run to run."""
    dev = require_cuda()
    wl = synth.workload(name, K=K)
    w, t = synth.head_weights(wl), synth.t_sched(wl.K)
    cond, noise = dev_bf16(synth.cond(wl)), dev_f32(synth.noise(wl))
    head = make_head(wl, w)
    S = int(round(wl.n * (1 - wl.filter_q)))
    idx = torch.randperm(wl.n, device=dev, generator=torch.Generator(device=dev).manual_seed(3))[:S]
    idx = idx.sort().values.to(torch.int32).contiguous()
    count = torch.tensor([S], dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    ref = None
    for r in range(runs):
        if r % 3 == 1:                                  # a different, smaller run in between
            c2 = torch.tensor([S // 2 + 7 * r], dtype=torch.int32, device=dev)
            scratch = torch.empty((wl.n, wl.C), dtype=torch.float32, device=dev)
            head.ardiff_head_sample(cond, noise, t, idx, c2, scratch)
        flush.fill_(r)
        out = torch.full((wl.n, wl.C), SENTINEL, dtype=torch.float32, device=dev)
        head.ardiff_head_sample(cond, noise, t, idx, count, out)
        assert head.status() == 0
        if ref is None:
            ref = out
        else:
            assert torch.equal(out, ref), f"run {r} differs from run 0"
    assert bool(torch.isfinite(ref[idx.long()]).all())
    head.close()


@pytest.mark.parametrize("name,extra,K", [("cfg2", 160, None), ("cfg3", 48, None), ("cfg4", 32, None),
                                          ("cfg3", 24, 1), ("cfg3", 12, 8)])
def test_workload_configs_sampled_tokens(name, extra, K):
    """Full-size gate -> head run; the oracle checks one token of every token tile, the first, a middle
    and the last (ragged) token tile and random survivors one by one (tokens are independent). cfg 3
    also runs at the other step counts its workload names (K = 1 and 8)."""
    dev = require_cuda()
    wl = synth.workload(name) if K is None else synth.workload(name, K=K)
    feat_bits = synth.features(wl)
    H = oracle.entropy(feat_bits)
    Hs = np.sort(H)
    k = int(round(wl.filter_q * wl.n))
    tau = 0.5 * (Hs[k - 1] + Hs[k])
    w, cond_bits, noise, t = synth.head_weights(wl), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K)
    head = make_head(wl, w)
    mask, idx, count, _ = ardiff.ardiff_entropy_gate(dev_bf16(feat_bits), tau)
    out = torch.full(noise.shape, SENTINEL, dtype=torch.float32, device=dev)
    head.ardiff_head_sample(dev_bf16(cond_bits), dev_f32(noise), t, idx, count, out)
    assert head.status() == 0
    S = int(count.item())
    idx_h = idx.cpu().numpy()[:S]
    got = out.cpu().numpy()
    # Oracle-checked, element by element: one random token of EVERY token tile (an error confined to some
    # tiles, a group boundary or a scratch-slot reuse cannot hide), plus the whole first, one middle and the
    # last (ragged) tile and some random survivors. At the other step counts of cfg 3 the whole tiles are
    # thinned to keep the oracle's share of the run to seconds.
    rng = np.random.default_rng(11)
    tiles = (S + 127) // 128
    per_tile = np.minimum(np.arange(tiles) * 128 + rng.integers(0, 128, size=tiles), S - 1)
    whole = sample_tokens(idx_h, extra=extra)
    if K is not None:
        whole = whole[::4]
    pos = np.unique(np.concatenate([per_tile, whole]))
    toks = idx_h[pos]
    want = oracle.head_sample(w, cond_bits, noise, t, toks)

    def floor(rows):        # what bf16 rounding alone costs these tokens (CPU model, fp64)
        exact = rounding_model.head(w, cond_bits, noise, t, rows, rounded=())
        return rounding_model.error_ratio(rounding_model.head(w, cond_bits, noise, t, rows), exact)

    assert_head_parity(got, want, toks, name, model=floor)
    # properties that hold for every token: written iff kept, finite
    kept = np.zeros(wl.n, bool)
    kept[idx_h] = True
    assert np.all(got[~kept] == SENTINEL)
    assert np.all(np.isfinite(got[kept])) and not np.any(got[kept] == SENTINEL)
    head.close()


def test_two_heads_on_two_streams():
    """Two heads of different shapes, driven from two streams without any ordering between them: every
    launch needs the whole GPU (cooperative launch), so the launches take turns; both results must
    match what each head gives alone."""
    dev = require_cuda()
    wa, wb = synth.workload("cfg1", n=700), synth.workload("cfg1", n=900, W=512, L=3, seed=77)
    outs = {}
    heads = {}
    for key, wl in (("a", wa), ("b", wb)):
        w, t = synth.head_weights(wl), synth.t_sched(wl.K)
        head = make_head(wl, w)
        cond, noise = dev_bf16(synth.cond(wl)), dev_f32(synth.noise(wl))
        idx = torch.arange(wl.n, dtype=torch.int32, device=dev)
        count = torch.tensor([wl.n], dtype=torch.int32, device=dev)
        alone = torch.empty((wl.n, wl.C), dtype=torch.float32, device=dev)
        head.ardiff_head_sample(cond, noise, t, idx, count, alone)
        heads[key] = (head, cond, noise, t, idx, count, alone, wl)
    torch.cuda.synchronize()
    streams = {k: torch.cuda.Stream(device=dev) for k in heads}
    for rep in range(4):
        for key, (head, cond, noise, t, idx, count, alone, wl) in heads.items():
            out = torch.full((wl.n, wl.C), SENTINEL, dtype=torch.float32, device=dev)
            head.ardiff_head_sample(cond, noise, t, idx, count, out, stream=streams[key])
            outs[(key, rep)] = out
    torch.cuda.synchronize()
    for (key, rep), out in outs.items():
        head, *_, alone, wl = heads[key]
        assert head.status() == 0
        assert torch.equal(out, alone), (key, rep)
    for head, *_ in heads.values():
        head.close()


def test_bad_arguments_are_rejected():
    require_cuda()
    wl = synth.workload("cfg1")
    w = synth.head_weights(wl)
    with pytest.raises(ardiff.ArdiffError):
        ardiff.Head(wl.C, wl.Dc, 250, wl.L, wl.F, 4, 64, w)          # W not a multiple of 256
    with pytest.raises(ardiff.ArdiffError):
        ardiff.Head(8, wl.Dc, wl.W, wl.L, wl.F, 4, 64, w)            # C too small
    head = make_head(wl, w)
    lib = ardiff.lib()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    p = buf.data_ptr()
    t = synth.t_sched(4)
    assert lib.ardiff_head_sample(head._h, p, p, t.ctypes.data, 5, p, p, p, None) == ardiff.ARDIFF_ERR_SHAPE
    assert lib.ardiff_head_sample(head._h, p, p, t.ctypes.data, 4, None, p, p, None) == ardiff.ARDIFF_ERR_NULL
    assert lib.ardiff_head_sample(head._h, p + 2, p, t.ctypes.data, 4, p, p, p, None) == ardiff.ARDIFF_ERR_ALIGN
    head.close()


def ddim_coef(abar):
    """Deterministic eps-prediction steps along abar[0] -> abar[1] -> ... (coefficients of x and eps)."""
    abar = np.asarray(abar, np.float64)
    ax = np.sqrt(abar[1:] / abar[:-1])
    av = np.sqrt(1 - abar[1:]) - ax * np.sqrt(1 - abar[:-1])
    return np.stack([ax, av, np.zeros_like(ax)], axis=1).astype(np.float32)


@pytest.mark.parametrize("sampler", ["euler", "ddim", "x0_renoise"])
def test_linear_sampler_steps(sampler):
    """Other samplers on the same head: every step is x <- ax x + av v + an z_k."""
    dev = require_cuda()
    wl = synth.workload("cfg1", n=300, K=4)
    # all three on the harder 1/sqrt(fan_in) weights (every layer keeps unit scale, nothing damps an error)
    w = synth.head_weights(wl, std=None)
    cond_bits, noise = synth.cond(wl), synth.noise(wl)
    idx_np = np.random.default_rng(7).permutation(wl.n)[:211].astype(np.int32)
    z = None
    if sampler == "euler":
        t = np.array([0.0, 0.2, 0.5, 0.9, 1.0], np.float32)
        t_in = t[:-1]
        coef = np.stack([np.ones(4), t[1:].astype(np.float64) - t[:-1].astype(np.float64), np.zeros(4)], 1).astype(np.float32)
    elif sampler == "ddim":
        t_in = np.array([0.95, 0.7, 0.45, 0.2], np.float32)
        coef = ddim_coef([0.05, 0.3, 0.6, 0.85, 0.999])
    else:
        # two-step consistency sampling: predict x0, re-noise to abar = 0.5, predict x0 again. The output
        # is the head's last raw prediction (ax = 0 discards the state), so nothing props up its RMS.
        t_in = np.array([0.95, 0.5], np.float32)
        abn = np.array([0.5, 1.0])
        coef = np.stack([np.zeros(2), np.sqrt(abn), np.sqrt(1 - abn)], 1).astype(np.float32)
        z = np.random.default_rng(8).standard_normal((2, wl.n, wl.C)).astype(np.float32)
    want = oracle.head_sample_coef(w, cond_bits, noise, t_in, coef, idx_np, step_noise=z)
    head = make_head(wl, w)
    idx = torch.from_numpy(idx_np).to(dev)
    count = torch.tensor([len(idx_np)], dtype=torch.int32, device=dev)
    out = torch.full(noise.shape, SENTINEL, dtype=torch.float32, device=dev)
    head.ardiff_head_sample_coef(dev_bf16(cond_bits), dev_f32(noise), t_in, coef, idx, count, out,
                                 step_noise=None if z is None else torch.from_numpy(z).to(dev))
    assert head.status() == 0
    got = out.cpu().numpy()
    assert_parity(got, want, idx_np, sampler)
    assert np.all(got[np.setdiff1d(np.arange(wl.n), idx_np)] == SENTINEL)
    if sampler == "euler":                 # the Euler entry point is this call with the Euler coefficients
        got2 = run_head(head, cond_bits, noise, np.array([0.0, 0.2, 0.5, 0.9, 1.0], np.float32), idx_np)
        assert np.array_equal(got2[idx_np], got[idx_np])
    head.close()


@pytest.mark.parametrize("shape", [dict(W=4096, L=1, K=1, C=32, Dc=64, n=130),
                                   dict(W=2048, L=2, K=2, C=64, Dc=128, n=300),
                                   dict(W=256, L=5, K=3, C=48, Dc=1024, n=257),
                                   dict(W=512, L=1, K=64, C=16, Dc=64, n=40),
                                   dict(W=256, L=64, K=1, C=16, Dc=64, n=130),
                                   dict(W=512, L=2, K=2, C=16, Dc=128, F=1024, n=200),
                                   dict(W=256, L=2, K=3, C=32, Dc=64, F=2, n=129)])
def test_extreme_shapes(shape):
    """Widest head (16 column tiles, 32 LayerNorm partials per row), the largest token dim, an odd number
    of blocks (gate buffers alternate by block parity), the largest step count, the deepest head (64 blocks),
    the largest and the smallest time-embedding size."""
    n = shape.pop("n")
    wl = synth.workload("cfg1", n=n, **shape)
    w, cond_bits, noise, t = synth.head_weights(wl), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K)
    idx = np.arange(n, dtype=np.int32)
    want = oracle.head_sample(w, cond_bits, noise, t, idx)
    head = make_head(wl, w)
    got = run_head(head, cond_bits, noise, t, idx)
    assert_parity(got, want, idx, str(shape))
    head.close()


def test_bounded_wait_runs_out_reports_timeout_and_the_head_recovers():
    """The self-test hook makes one tile's dependency wait unsatisfiable and shortens the wait limit to 3 ms:
    the kernel must come back by itself (no fault, no trap, no endless spin), the status word must say
    TIMEOUT, and the very next call on the same head must give the bits of an undisturbed run."""
    wl = synth.workload("cfg1", n=900)
    w, cond_bits, noise, t = synth.head_weights(wl), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K)
    idx = np.arange(wl.n, dtype=np.int32)
    head = make_head(wl, w)
    clean = run_head(head, cond_bits, noise, t, idx)
    for tile in (0, 3, 7):                                # first, an odd (partner CTA) and the last, ragged tile
        head.inject_stall(tile, 3000)
        dev = require_cuda()
        out = torch.zeros(noise.shape, dtype=torch.float32, device=dev)
        head.ardiff_head_sample(dev_bf16(cond_bits), dev_f32(noise), t, torch.from_numpy(idx).to(dev),
                                torch.tensor([wl.n], dtype=torch.int32, device=dev), out)
        assert head.status() == ardiff.ARDIFF_ERR_TIMEOUT
        assert head.status() == 0                         # reading the status clears it
        assert np.array_equal(run_head(head, cond_bits, noise, t, idx), clean)
    head.inject_stall(4000, 3000)                         # a tile this call does not have: no effect
    assert np.array_equal(run_head(head, cond_bits, noise, t, idx), clean)
    fresh = make_head(wl, w)
    assert np.array_equal(run_head(fresh, cond_bits, noise, t, idx), clean)
    with pytest.raises(ardiff.ArdiffError):
        head.inject_stall(0, 5)                           # limit below 100 us
    fresh.close()
    head.close()


def test_more_survivors_than_the_head_was_created_for():
    """*count above max_tokens: the head runs the first max_tokens survivors, leaves every other row
    untouched and flags the call with ARDIFF_ERR_SHAPE in its status word; the next call is clean."""
    dev = require_cuda()
    wl = synth.workload("cfg1", n=400)
    w, cond_bits, noise, t = synth.head_weights(wl), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K)
    head = make_head(wl, w, max_tokens=256)
    idx_np = np.random.default_rng(2).permutation(wl.n)[:300].astype(np.int32)
    want = oracle.head_sample(w, cond_bits, noise, t, idx_np[:256])
    idx = torch.from_numpy(idx_np).to(dev)
    count = torch.tensor([300], dtype=torch.int32, device=dev)
    out = torch.full(noise.shape, SENTINEL, dtype=torch.float32, device=dev)
    head.ardiff_head_sample(dev_bf16(cond_bits), dev_f32(noise), t, idx, count, out)
    assert head.status() == ardiff.ARDIFF_ERR_SHAPE
    got = out.cpu().numpy()
    assert_parity(got, want, idx_np[:256])
    assert np.all(got[np.setdiff1d(np.arange(wl.n), idx_np[:256])] == SENTINEL)
    assert np.array_equal(run_head(head, cond_bits, noise, t, idx_np[:200])[idx_np[:200]], got[idx_np[:200]])
    head.close()


def test_persisting_l2_is_set_aside_while_a_head_exists_and_put_back_after():
    # include/ardiff.h, ardiff_head_create: the context's persisting-L2 limit covers one token group's fp32
    # residual stream while heads exist on the device, and returns to what it was with the last of them
    rt = pytest.importorskip("cuda.bindings.runtime")
    require_cuda()

    def limit():
        err, v = rt.cudaDeviceGetLimit(rt.cudaLimit.cudaLimitPersistingL2CacheSize)
        assert int(err) == 0
        return int(v)

    err, max_size = rt.cudaDeviceGetAttribute(rt.cudaDeviceAttr.cudaDevAttrMaxPersistingL2CacheSize, 0)
    assert int(err) == 0
    if max_size <= 0:
        pytest.skip("device has no persisting L2")
    wl = synth.workload("cfg1")
    weights = synth.head_weights(wl)
    before = limit()
    h1 = make_head(wl, weights)
    during = limit()
    group_h_bytes = 2 * 128 * wl.W * 4          # cfg1: one pair of token tiles per group
    assert during >= min(group_h_bytes, max_size) and during >= before
    h2 = make_head(wl, weights)
    h1.close()
    assert limit() == during
    h2.close()
    assert limit() == before
