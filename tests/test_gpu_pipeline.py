"""GPU tests of the host-buffer front end (ardiff_pipeline_*): the blocking call against the fp64
oracle, and the overlapped submit / wait / join calls against the blocking call on the same batches.

Agreement bars: as in the gate and head tests (mask equal outside a 1e-4 entropy band around tau,
per token max |out - oracle| <= 2e-2 * RMS(oracle row)); overlapped vs blocking: bit-exact, since
both run the same kernels on the same data.
"""
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
    one.close()
    two.close()
    head.close()
