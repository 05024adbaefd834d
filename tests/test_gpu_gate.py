"""GPU parity of the entropy gate + compaction against the fp64 oracle, through the C ABI.

Agreement bar: entropy within 1e-3 absolute; mask equal for every token whose oracle entropy is
at least 1e-4 away from tau; idx/count bit-exact against the GPU's own mask (ascending positions)
and, when no token lies in the band, bit-exact against the oracle's.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2512_08537_b200 as ardiff
from gpu_util import dev_bf16, require_cuda

pytestmark = pytest.mark.gpu

ENT_TOL = 1e-3
BAND = 1e-4


def run_gate(bits, tau):
    feat = dev_bf16(bits)
    mask, idx, count, ent = ardiff.ardiff_entropy_gate(feat, tau, want_entropy=True)
    torch.cuda.synchronize()
    c = int(count.item())
    return mask.cpu().numpy(), idx.cpu().numpy()[:c], c, ent.cpu().numpy()


def check(bits, tau):
    H, mask_o, idx_o, count_o = oracle.gate(bits, tau)
    mask_g, idx_g, count_g, ent_g = run_gate(bits, tau)
    nan_o = np.isnan(H)
    assert np.array_equal(np.isnan(ent_g), nan_o)
    assert np.all(np.abs(ent_g[~nan_o] - H[~nan_o]) <= ENT_TOL)
    off_band = nan_o | (np.abs(H - float(np.float32(tau))) >= BAND)
    assert np.array_equal(mask_g[off_band], mask_o[off_band])
    assert count_g == int(mask_g.sum())
    assert np.array_equal(idx_g, np.flatnonzero(mask_g).astype(np.int32))
    if off_band.all():
        assert count_g == count_o and np.array_equal(idx_g, idx_o)
    return H, mask_g, count_g


def quantile_tau(H, q):
    """Midpoint between neighbouring order statistics, so the band around tau is usually empty."""
    Hs = np.sort(H[~np.isnan(H)])
    k = int(round(q * len(Hs)))
    if k <= 0:
        return -1.0
    if k >= len(Hs):
        return float(Hs[-1]) + 1.0
    return 0.5 * (float(Hs[k - 1]) + float(Hs[k]))


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4"])
def test_workload_configs(name):
    wl = synth.workload(name)
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    tau = quantile_tau(H, wl.filter_q)
    _, mask_g, count_g = check(bits, tau)
    assert abs(count_g - round((1 - wl.filter_q) * wl.n)) <= 16


@pytest.mark.parametrize("n", [1, 7, 8, 31, 33, 129, 1000, 4099])
@pytest.mark.parametrize("d", [8, 16, 256, 264, 768, 1024, 2048, 3072, 5120, 6144, 8192])
def test_shapes_vector_path(n, d):
    if n * d > 4099 * 1024 and n > 129:
        n = 129
    wl = synth.workload("cfg2", n=n, d=d, seed=1000 + d)
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    for q in (0.0, 0.5, 1.0):
        check(bits, quantile_tau(H, q))


@pytest.mark.parametrize("d", [8200, 12288, 16384, 65536])
def test_shapes_long_rows_single_pass(d):
    """Rows longer than the registers hold (d > 8192, d % 8 == 0): one pass with a running maximum per lane."""
    wl = synth.workload("cfg4", n=41, d=d, seed=3000 + d)
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    for q in (0.0, 0.4):
        check(bits, quantile_tau(H, q))
    x = np.zeros((3, d), np.float32)
    x[0, d - 5] = 90.0                    # the maximum arrives at the very end: every partial sum is rescaled
    x[1, :d // 2] = -np.inf               # -inf channels contribute nothing
    x[2, 4000] = np.nan                   # dropped
    Hs, mask_g, _ = check(synth.f32_to_bf16(x), 0.5)
    assert list(mask_g) == [0, 1, 0] and abs(Hs[1] - np.log(d - d // 2)) < 1e-9


@pytest.mark.parametrize("d", [1, 2, 7, 12, 777, 1001, 8201, 16383])
def test_shapes_generic_path(d):
    wl = synth.workload("cfg2", n=67, d=d, seed=2000 + d)
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    for q in (0.0, 0.4):
        check(bits, quantile_tau(H, q))


def test_empty_input_writes_zero_count():
    dev = require_cuda()
    feat = torch.empty((0, 64), dtype=torch.bfloat16, device=dev)
    count = torch.full((1,), 77, dtype=torch.int32, device=dev)
    ardiff.ardiff_entropy_gate(feat, 0.5, count=count)
    torch.cuda.synchronize()
    assert int(count.item()) == 0


def test_special_rows_minus_inf_nan_inf_uniform_onehot():
    d = 512
    x = np.zeros((8, d), np.float32)
    x[1, 5] = 100.0                       # one-hot limit -> 0
    x[2, :100] = -np.inf                  # -inf channels contribute nothing: H = ln(412)
    x[3, :] = -np.inf                     # undefined -> dropped
    x[4, 17] = np.nan                     # dropped
    x[5, 300] = np.inf                    # dropped
    x[6, :] = 3.0                         # uniform: ln d
    x[7, ::2] = 1.5                       # two-level closed form
    bits = synth.f32_to_bf16(x)
    H, mask_g, count_g = check(bits, 0.5)
    assert abs(H[0] - np.log(d)) < 1e-12 and abs(H[2] - np.log(412)) < 1e-12
    assert list(mask_g) == [1, 0, 1, 0, 0, 0, 1, 1]
    # same rows through the generic kernel (d not a multiple of 8)
    check(synth.f32_to_bf16(x[:, :509]), 0.5)


def test_tau_extremes_keep_all_and_drop_all():
    wl = synth.workload("cfg2", n=3000)
    bits = synth.features(wl)
    _, m_all, c_all = check(bits, -1.0)
    assert c_all == 3000
    _, m_none, c_none = check(bits, 100.0)
    assert c_none == 0


def test_bad_arguments_are_rejected_without_launching():
    dev = require_cuda()
    lib = ardiff.lib()
    buf = torch.zeros(4096, dtype=torch.uint8, device=dev)
    p = buf.data_ptr()
    assert lib.ardiff_entropy_gate(None, 4, 8, 0.0, p, p, p, None) == ardiff.ARDIFF_ERR_NULL
    assert lib.ardiff_entropy_gate(p, 4, 8, 0.0, p, p, None, None) == ardiff.ARDIFF_ERR_NULL
    assert lib.ardiff_entropy_gate(p, -1, 8, 0.0, p, p, p, None) == ardiff.ARDIFF_ERR_SHAPE
    assert lib.ardiff_entropy_gate(p, 4, 0, 0.0, p, p, p, None) == ardiff.ARDIFF_ERR_SHAPE
    assert lib.ardiff_entropy_gate(p + 2, 4, 8, 0.0, p, p, p, None) == ardiff.ARDIFF_ERR_ALIGN
    torch.cuda.synchronize()


def test_gate_calls_on_two_unordered_streams():
    """Two gate calls of different shapes enqueued on two streams with no ordering between them (they may
    overlap on the GPU: each stream has its own block-count scratch) give what each gives alone."""
    dev = require_cuda()
    jobs = {}
    for key, (n, d, q) in {"a": (60000, 768, 0.3), "b": (9001, 5120, 0.6)}.items():
        wl = synth.workload("cfg2" if key == "a" else "cfg4", n=n, d=d)
        feat = dev_bf16(synth.features(wl))
        _, _, _, ent = ardiff.ardiff_entropy_gate(feat, -1.0, want_entropy=True)
        tau = float(np.quantile(ent.cpu().numpy(), q))
        mask, idx, count, _ = ardiff.ardiff_entropy_gate(feat, tau)
        torch.cuda.synchronize()
        jobs[key] = (feat, tau, mask.clone(), idx.clone(), int(count.item()))
    streams = {k: torch.cuda.Stream(device=dev) for k in jobs}
    res = []
    for rep in range(6):
        for key, (feat, tau, *_rest) in jobs.items():
            with torch.cuda.stream(streams[key]):
                m, i, c, _ = ardiff.ardiff_entropy_gate(feat, tau, stream=streams[key])
            res.append((key, m, i, c))
    torch.cuda.synchronize()
    for key, m, i, c in res:
        _, _, mask, idx, count = jobs[key]
        assert int(c.item()) == count and torch.equal(m, mask) and torch.equal(i[:count], idx[:count]), key


def test_full_size_gate_stress_sampled_rows_and_properties():
    """2^20 x 5120 (10.7 GB): features are generated and uploaded in slabs; the oracle checks a
    sample of rows one by one, the rest is checked through properties that hold at any size."""
    dev = require_cuda()
    wl = synth.workload("cfg5")
    free, _ = torch.cuda.mem_get_info()
    if free < 14 * 2**30:
        pytest.fail("needs 14 GB of free device memory")
    feat = torch.empty((wl.n, wl.d), dtype=torch.bfloat16, device=dev)
    slab = 32768
    for r0 in range(0, wl.n, slab):
        feat[r0:r0 + slab] = dev_bf16(synth.features(wl, r0, slab))
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([np.arange(0, 64), np.arange(wl.n - 64, wl.n),
                                     rng.integers(0, wl.n, size=4096)]))
    H_s = np.array([oracle.entropy(synth.features(wl, int(r), 1))[0] for r in rows])
    cond = torch.empty((wl.n, wl.Dc), dtype=torch.bfloat16, device=dev)
    noise = torch.empty((wl.n, wl.C), dtype=torch.float32, device=dev)
    big = 1 << 17
    for r0 in range(0, wl.n, big):
        cond[r0:r0 + big] = dev_bf16(synth.cond(wl, r0, big))
        noise[r0:r0 + big] = torch.from_numpy(synth.noise(wl, r0, big)).to(dev)
    w, t = synth.head_weights(wl), synth.t_sched(wl.K)
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, wl.n, w)
    out = torch.empty((wl.n, wl.C), dtype=torch.float32, device=dev)
    for q in (0.0, 0.1, 0.5, 0.9, 0.99):
        tau = quantile_tau(H_s, q)
        mask, idx, count, ent = ardiff.ardiff_entropy_gate(feat, tau, want_entropy=True)
        torch.cuda.synchronize()
        c = int(count.item())
        ent_s = ent[torch.from_numpy(rows).to(dev)].cpu().numpy()
        mask_s = mask[torch.from_numpy(rows).to(dev)].cpu().numpy()
        assert np.all(np.abs(ent_s - H_s) <= ENT_TOL)
        off = np.abs(H_s - float(np.float32(tau))) >= BAND
        assert np.array_equal(mask_s[off], (H_s >= float(np.float32(tau))).astype(np.uint8)[off])
        assert c == int(mask.sum().item())
        want_idx = torch.nonzero(mask, as_tuple=False).flatten().to(torch.int32)
        assert torch.equal(idx[:c], want_idx)
        assert abs(c / wl.n - (1 - q)) < 0.03
        if q == 0.1:
            continue                                   # head runs: 0, 50, 90 and 99 % filtered
        # The survivors feed the cfg2-shaped head: from 8192 token tiles with the scratch ring wrapping many
        # times (0 %) to an under-filled grid with a ragged tail (99 %). The oracle checks, one by one, every
        # third token of the first tile, the whole last (ragged) tile and one random token of every 16th tile.
        S = c
        idx_h = idx[:S].cpu().numpy()
        out.fill_(-777.0)
        head.ardiff_head_sample(cond, noise, t, idx, count, out)
        assert head.status() == 0
        tiles = (S + 127) // 128
        pos = np.concatenate([np.arange(0, min(S, 128), 3), np.arange(max(0, S - (S % 128 or 128)), S),
                              np.arange(0, tiles, 16) * 128 + rng.integers(0, 128, size=len(range(0, tiles, 16)))])
        pos = np.unique(pos[pos < S])
        toks = idx_h[pos]
        cond_s = np.concatenate([synth.cond(wl, int(tk), 1) for tk in toks])
        noise_s = np.concatenate([synth.noise(wl, int(tk), 1) for tk in toks])
        want = oracle.head_sample(w, cond_s, noise_s, t, np.arange(len(toks), dtype=np.int32))
        got = out[torch.from_numpy(toks.astype(np.int64)).to(dev)].cpu().numpy().astype(np.float64)
        err = np.abs(got - want).max(axis=1) / np.sqrt((want ** 2).mean(axis=1))
        assert err.max() <= 2e-2, (q, err.max())
        written = (out[:, 0] != -777.0)                # written iff kept, and finite
        assert int(written.sum().item()) == S and torch.equal(written, mask.bool())
        assert bool(torch.isfinite(out[written]).all())
    head.close()
