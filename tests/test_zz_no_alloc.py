"""ardiff_entropy_gate_noalloc against ardiff_entropy_gate, through the C ABI.

The no-alloc entry point exists for callers that must not let a library allocate device memory
(an application whose own pool owns the GPU, work issued during a stream capture, a real-time
loop). It runs the same kernels as the regular gate with its per-block scratch taken from a fixed
__device__ array inside the library, so its outputs must match the regular entry point bit for
bit. The array is shared by all calls and keeps what the last call wrote: the test therefore makes
two calls in a row with different shapes and thresholds (the second with fewer blocks than the
first, so stale entries are present) and checks both. This file sorts last on purpose: a run that
stops at the first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import synth
import paper_2512_08537_b200 as ardiff
from gpu_util import dev_bf16, require_cuda

pytestmark = pytest.mark.gpu


def _both(feat, tau):
    dev = feat.device
    n = feat.shape[0]
    mask_a, idx_a, count_a, _ = ardiff.ardiff_entropy_gate(feat, tau)
    mask_b = torch.full((n,), 7, dtype=torch.uint8, device=dev)
    idx_b = torch.full((n,), -5, dtype=torch.int32, device=dev)
    count_b = torch.full((1,), -1, dtype=torch.int32, device=dev)
    ardiff.ardiff_entropy_gate_noalloc(feat, tau, mask_b, idx_b, count_b)
    torch.cuda.synchronize()
    ca, cb = int(count_a.item()), int(count_b.item())
    assert ca == cb
    assert torch.equal(mask_a, mask_b)
    assert torch.equal(idx_a[:ca], idx_b[:cb])
    assert torch.all(idx_b[cb:] == -5)              # nothing is written past count
    return ca


def test_noalloc_gate_matches_regular_gate_on_two_calls_in_a_row():
    require_cuda()
    # call 1: many blocks (every entry of the fixed array that a launch can use gets written)
    wl = synth.workload("cfg2", n=40000)
    bits = synth.features(wl)
    feat1 = dev_bf16(bits)
    _, _, _, ent = ardiff.ardiff_entropy_gate(feat1, -1.0, want_entropy=True)
    tau1 = float(np.median(ent.cpu().numpy()))
    kept1 = _both(feat1, tau1)
    assert 0 < kept1 < wl.n
    # call 2, straight after: a ragged, much smaller input with another width and threshold
    wl2 = synth.workload("cfg4", n=1003)
    feat2 = dev_bf16(synth.features(wl2))
    _, _, _, ent2 = ardiff.ardiff_entropy_gate(feat2, -1.0, want_entropy=True)
    tau2 = float(np.quantile(ent2.cpu().numpy(), 0.3))
    kept2 = _both(feat2, tau2)
    assert 0 < kept2 < wl2.n
    # and the first input again: the result does not depend on what is left in the array
    assert _both(feat1, tau1) == kept1


def test_noalloc_gate_leaves_device_memory_as_it_found_it():
    """What the entry point is for: after its first call on the device (symbol look-up, kernel load), a call
    takes no device memory: the driver's count of free bytes is the same before and after."""
    require_cuda()
    wl = synth.workload("cfg2", n=5000)
    feat = dev_bf16(synth.features(wl))
    dev = feat.device
    mask = torch.empty((wl.n,), dtype=torch.uint8, device=dev)
    idx = torch.empty((wl.n,), dtype=torch.int32, device=dev)
    count = torch.empty((1,), dtype=torch.int32, device=dev)
    ardiff.ardiff_entropy_gate_noalloc(feat, 5.0, mask, idx, count)          # first call for this row width
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for n in (5000, 1234):
        ardiff.ardiff_entropy_gate_noalloc(feat[:n], 5.0, mask, idx, count)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_noalloc_gate_rejects_sizes_beyond_its_fixed_capacity_and_handles_empty_input():
    dev = require_cuda()
    lib = ardiff.lib()
    fn = lib.ardiff_entropy_gate_noalloc
    vp = ctypes.c_void_p
    fn.restype = ctypes.c_int
    fn.argtypes = [vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_float, vp, vp, vp, vp]
    buf = torch.zeros(4096, dtype=torch.uint8, device=dev)
    p = buf.data_ptr()
    too_many = ardiff.GATE_NOALLOC_MAX_TOKENS + 1
    assert fn(p, too_many, 8, 0.0, p, p, p, None) == ardiff.ARDIFF_ERR_SHAPE   # nothing launched
    assert fn(p, -1, 8, 0.0, p, p, p, None) == ardiff.ARDIFF_ERR_SHAPE
    count = torch.full((1,), 9, dtype=torch.int32, device=dev)
    assert fn(None, 0, 8, 0.0, None, None, count.data_ptr(), None) == ardiff.ARDIFF_OK
    torch.cuda.synchronize()
    assert int(count.item()) == 0
