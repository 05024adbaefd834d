"""GPU tests of the host-buffer front end (ardiff_pipeline_*): the blocking call against the fp64
oracle, and the overlapped submit / wait / join calls against the blocking call on the same batches.

Agreement bars: as in the gate and head tests (mask equal outside a 1e-4 entropy band around tau,
per token max |out - oracle| <= 2e-2 * RMS(oracle row)); overlapped vs blocking: bit-exact, since
both run the same kernels on the same data.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2512_08537_b200 as ardiff
from gpu_util import require_cuda

pytestmark = pytest.mark.gpu

REL_TOL = 2e-2
BAND = 1e-4


def host_bf16(bits, pin=True):
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.pin_memory() if pin else t


def host_f32(x, pin=True):
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.pin_memory() if pin else t


def batch(wl, seed, n, pin=True):
    b = synth.workload(wl.name, n=n, seed=seed)
    g = synth.workload(wl.name, n=max(n, 1), seed=seed)     # an empty batch still passes valid pointers
    return (b, host_bf16(synth.features(g), pin)[:n], host_bf16(synth.cond(g), pin)[:n],
            host_f32(synth.noise(g), pin)[:n])


def outputs(n, C, pin=True):
    out = torch.full((max(n, 1), C), -5.0, dtype=torch.float32)
    mask = torch.full((max(n, 1),), 9, dtype=torch.uint8)
    if pin:
        out, mask = out.pin_memory(), mask.pin_memory()
    return out[:n], mask[:n]


@pytest.mark.parametrize("pin", [True, False])
def test_run_host_against_oracle(pin):
    require_cuda()
    wl = synth.workload("cfg1")
    w, t = synth.head_weights(wl), synth.t_sched(wl.K)
    b, feat, cond, noise = batch(wl, 11, 333, pin)
    feat_bits, cond_bits, noise_np = synth.features(b), synth.cond(b), synth.noise(b)
    H = oracle.entropy(feat_bits)
    tau = float(np.median(H))
    _, mask_o, idx_o, count_o = oracle.gate(feat_bits, tau)
    want = oracle.head_sample(w, cond_bits, noise_np, t, idx_o)
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, 512, w)
    pipe = ardiff.Pipeline(head, 512, wl.d)
    out, mask = outputs(b.n, wl.C, pin)
    kept = pipe.ardiff_pipeline_run_host(feat, cond, noise, tau, t, out, mask)
    assert head.status() == 0
    got, mask_g = out.numpy(), mask.numpy()
    off_band = np.abs(H - float(np.float32(tau))) >= BAND
    assert np.array_equal(mask_g[off_band], mask_o[off_band])
    assert kept == int(mask_g.sum())
    both = np.flatnonzero((mask_g == 1) & (mask_o == 1))
    err = np.abs(got[both].astype(np.float64) - want[both]).max(axis=1) / np.sqrt((want[both] ** 2).mean(axis=1))
    assert err.max() <= REL_TOL
    assert np.all(got[mask_g == 0] == 0.0)           # rows of dropped tokens are zero in the host result
    pipe.close()
    head.close()


def test_overlapped_batches_match_blocking_call():
    dev = require_cuda()
    wl = synth.workload("cfg1")
    w, t = synth.head_weights(wl), synth.t_sched(wl.K)
    max_n = 700
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, max_n, w)
    ref_pipe = ardiff.Pipeline(head, max_n, wl.d)
    pipe = ardiff.Pipeline(head, max_n, wl.d, slots=2)
    sizes = [700, 129, 0, 513, 1, 640, 700]          # ragged, empty and full batches through two slots
    taus = [5.0, 5.3, 5.0, -1.0, 5.2, 100.0, 5.25]   # -1 keeps everything, 100 drops everything
    batches = [batch(wl, 100 + i, n) for i, n in enumerate(sizes)]
    want = []
    for (b, feat, cond, noise), tau in zip(batches, taus):
        out, mask = outputs(b.n, wl.C)
        kept = ref_pipe.ardiff_pipeline_run_host(feat, cond, noise, tau, t, out, mask)
        want.append((out.clone(), mask.clone(), kept))
    assert 0 < want[0][2] < 700 and want[3][2] == 513 and want[5][2] == 0
    stream = torch.cuda.Stream(device=dev)
    outs = [outputs(b.n, wl.C) for b, *_ in batches]
    kept = [None] * len(batches)
    for i, ((b, feat, cond, noise), tau) in enumerate(zip(batches, taus)):
        slot = i % 2
        if i >= 2:
            kept[i - 2] = pipe.ardiff_pipeline_wait(slot)
        pipe.ardiff_pipeline_submit(slot, feat, cond, noise, tau, t, outs[i][0], outs[i][1], stream=stream)
    kept[-2] = pipe.ardiff_pipeline_wait((len(batches) - 2) % 2)
    kept[-1] = pipe.ardiff_pipeline_wait((len(batches) - 1) % 2)
    assert head.status() == 0
    for i in range(len(batches)):
        assert kept[i] == want[i][2], i
        assert torch.equal(outs[i][1], want[i][1]), i
        assert torch.equal(outs[i][0], want[i][0]), i
    # the blocking call still works on a multi-slot pipeline, and waiting twice is harmless
    b, feat, cond, noise = batches[0]
    out, mask = outputs(b.n, wl.C)
    assert pipe.ardiff_pipeline_run_host(feat, cond, noise, taus[0], t, out, mask) == want[0][2]
    assert torch.equal(out, want[0][0])
    assert pipe.ardiff_pipeline_wait(0) in (want[-1][2], want[-2][2])
    pipe.close()
    ref_pipe.close()
    head.close()


def test_run_host_while_another_slot_is_in_flight():
    """The blocking call on a multi-slot pipeline while a batch submitted on another slot may still be
    running: both use the one head, so the blocking call has to order itself after that batch. Both
    results must equal what the blocking call gives alone."""
    dev = require_cuda()
    wl = synth.workload("cfg1")
    w, t = synth.head_weights(wl), synth.t_sched(wl.K)
    max_n = 4096
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, max_n, w)
    ref_pipe = ardiff.Pipeline(head, max_n, wl.d)
    pipe = ardiff.Pipeline(head, max_n, wl.d, slots=3)
    ba, bb = batch(wl, 301, 4096), batch(wl, 302, 3001)
    want = []
    for b, feat, cond, noise in (ba, bb):
        out, mask = outputs(b.n, wl.C)
        kept = ref_pipe.ardiff_pipeline_run_host(feat, cond, noise, 5.1, t, out, mask)
        want.append((out.clone(), mask.clone(), kept))
    stream = torch.cuda.Stream(device=dev)
    for rep in range(3):
        oa, ma = outputs(ba[0].n, wl.C)
        ob, mb = outputs(bb[0].n, wl.C)
        pipe.ardiff_pipeline_submit(1, ba[1], ba[2], ba[3], 5.1, t, oa, ma, stream=stream)
        kept_b = pipe.ardiff_pipeline_run_host(bb[1], bb[2], bb[3], 5.1, t, ob, mb, stream=stream)   # no wait first
        kept_a = pipe.ardiff_pipeline_wait(1)
        assert head.status() == 0
        assert (kept_a, kept_b) == (want[0][2], want[1][2])
        assert torch.equal(oa, want[0][0]) and torch.equal(ma, want[0][1])
        assert torch.equal(ob, want[1][0]) and torch.equal(mb, want[1][1])
    pipe.close()
    ref_pipe.close()
    head.close()


def test_full_cfg2_through_three_slots_against_oracle():
    """The size the end-to-end figure is quoted on: 16384-token batches of the cfg 2 shape streamed through
    three slots; mask against the oracle outside the band, sampled survivors of every batch one by one."""
    require_cuda()
    wl = synth.workload("cfg2")
    w, t = synth.head_weights(wl), synth.t_sched(wl.K)
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, wl.n, w)
    pipe = ardiff.Pipeline(head, wl.n, wl.d, slots=3)
    n_batches = 5
    batches = [batch(wl, 400 + i, wl.n) for i in range(n_batches)]
    res = [outputs(wl.n, wl.C) for _ in range(n_batches)]
    taus, kept = [], [None] * n_batches
    for b, *_ in batches:
        H = oracle.entropy(synth.features(b))
        Hs = np.sort(H)
        k = int(round(wl.filter_q * wl.n))
        taus.append((0.5 * (Hs[k - 1] + Hs[k]), H))
    for i, (b, feat, cond, noise) in enumerate(batches):
        slot = i % 3
        if i >= 3:
            kept[i - 3] = pipe.ardiff_pipeline_wait(slot)
        pipe.ardiff_pipeline_submit(slot, feat, cond, noise, taus[i][0], t, res[i][0], res[i][1])
    for i in range(n_batches - 3, n_batches):
        kept[i] = pipe.ardiff_pipeline_wait(i % 3)
    assert head.status() == 0
    rng = np.random.default_rng(3)
    for i, (b, feat, cond, noise) in enumerate(batches):
        tau, H = taus[i]
        mask_o = (H >= float(np.float32(tau))).astype(np.uint8)
        got, mask_g = res[i][0].numpy(), res[i][1].numpy()
        off_band = np.abs(H - float(np.float32(tau))) >= BAND
        assert np.array_equal(mask_g[off_band], mask_o[off_band]) and kept[i] == int(mask_g.sum())
        surv = np.flatnonzero(mask_g)
        tiles = (len(surv) + 127) // 128
        pos = np.unique(np.minimum(np.arange(tiles) * 128 + rng.integers(0, 128, size=tiles), len(surv) - 1))
        toks = surv[pos]
        want = oracle.head_sample(w, synth.cond(b), synth.noise(b), t, toks.astype(np.int32))
        err = np.abs(got[toks].astype(np.float64) - want[toks]).max(axis=1) / np.sqrt((want[toks] ** 2).mean(axis=1))
        assert err.max() <= REL_TOL, (i, err.max())
        assert np.all(got[mask_g == 0] == 0.0) and np.all(np.isfinite(got))
    pipe.close()
    head.close()


def test_join_orders_a_stream_after_the_batches():
    dev = require_cuda()
    wl = synth.workload("cfg1")
    w, t = synth.head_weights(wl), synth.t_sched(wl.K)
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, 512, w)
    pipe = ardiff.Pipeline(head, 512, wl.d, slots=3)
    stream = torch.cuda.Stream(device=dev)
    res = []
    for s in range(3):
        b, feat, cond, noise = batch(wl, 200 + s, 400 + s)
        out, mask = outputs(b.n, wl.C)
        pipe.ardiff_pipeline_submit(s, feat, cond, noise, 5.0, t, out, mask, stream=stream)
        res.append((feat, cond, noise, out, mask))
    pipe.ardiff_pipeline_join(stream)
    stream.synchronize()                               # no ardiff_pipeline_wait: the join carries the order
    for feat, cond, noise, out, mask in res:
        m = mask.numpy()
        assert set(np.unique(m)) <= {0, 1}
        assert np.all(out.numpy()[m == 0] == 0.0) and np.all(np.isfinite(out.numpy()))
        assert np.all(out.numpy()[m == 1, 0] != -5.0)
    assert head.status() == 0
    pipe.close()
    head.close()


def test_bad_arguments():
    require_cuda()
    wl = synth.workload("cfg1")
    w, t = synth.head_weights(wl), synth.t_sched(wl.K)
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, 256, w)
    lib = ardiff.lib()
    one = ardiff.Pipeline(head, 256, wl.d)
    two = ardiff.Pipeline(head, 256, wl.d, slots=2)
    b, feat, cond, noise = batch(wl, 1, 300)
    out, mask = outputs(b.n, wl.C)
    with pytest.raises(RuntimeError):
        one.ardiff_pipeline_submit(0, feat[:8], cond[:8], noise[:8], 5.0, t, out[:8], mask[:8])
    with pytest.raises(RuntimeError):
        one.ardiff_pipeline_join()
    with pytest.raises(RuntimeError):                  # more tokens than the staging buffers hold
        two.ardiff_pipeline_submit(0, feat, cond, noise, 5.0, t, out, mask)
    with pytest.raises(RuntimeError):
        two.ardiff_pipeline_run_host(feat, cond, noise, 5.0, t, out, mask)
    with pytest.raises(ValueError):
        two.ardiff_pipeline_submit(2, feat[:8], cond[:8], noise[:8], 5.0, t, out[:8], mask[:8])
    assert lib.ardiff_pipeline_wait(two._p, 5) == ardiff.ARDIFF_ERR_SHAPE
    assert lib.ardiff_pipeline_wait(None, 0) == ardiff.ARDIFF_ERR_NULL
    assert two.ardiff_pipeline_wait(1) == 0            # never submitted: returns at once
    with pytest.raises(RuntimeError):
        ardiff.Pipeline(head, 256, wl.d, slots=5)
    # staging buffers that do not match the head: more tokens than it can run, another cond width or token dim
    vp = ctypes.c_void_p
    create = lib.ardiff_pipeline_create_slots
    h = ctypes.c_void_p()
    assert create(head._h, 257, wl.d, wl.Dc, wl.C, 1, ctypes.byref(h)) == ardiff.ARDIFF_ERR_SHAPE
    assert create(head._h, 256, wl.d, wl.Dc + 64, wl.C, 1, ctypes.byref(h)) == ardiff.ARDIFF_ERR_SHAPE
    assert create(head._h, 256, wl.d, wl.Dc, wl.C + 16, 1, ctypes.byref(h)) == ardiff.ARDIFF_ERR_SHAPE
    one.close()
    two.close()
    head.close()
