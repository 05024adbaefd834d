"""Python binding of libardiff (the C ABI declared in include/ardiff.h).

Argument marshalling only: every step of the hot path runs in the CUDA kernels of the shared
library. torch is used for device memory and streams. There is no CPU fallback: if the library
cannot be loaded, or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libardiff.so")
_lib = None

ARDIFF_OK = 0
ARDIFF_ERR_NULL, ARDIFF_ERR_SHAPE, ARDIFF_ERR_ALIGN, ARDIFF_ERR_UNSUPPORTED = -1, -2, -3, -4
ARDIFF_ERR_CUDA, ARDIFF_ERR_TIMEOUT, ARDIFF_ERR_NOMEM = -5, -6, -7

_WEIGHT_FIELDS = ["Wc", "bc", "Wt1", "bt1", "Wt2", "bt2", "Win", "bin", "Wmod", "bmod",
                  "W1", "b1", "W2", "b2", "Wfm", "bfm", "Wout", "bout"]


class ArdiffError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class HeadDesc(ctypes.Structure):
    _fields_ = [("C", ctypes.c_int32), ("Dc", ctypes.c_int32), ("W", ctypes.c_int32),
                ("L", ctypes.c_int32), ("F", ctypes.c_int32), ("K_max", ctypes.c_int32),
                ("max_tokens", ctypes.c_int64)]


class HeadHostWeights(ctypes.Structure):
    _fields_ = [(k, ctypes.c_void_p) for k in _WEIGHT_FIELDS]


def lib() -> ctypes.CDLL:
    """Loads libardiff.so (building it with nvcc first if it is missing). Raises if it cannot."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            from . import build as _build
            _build.build()
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float
        L.ardiff_strerror.restype = ctypes.c_char_p
        L.ardiff_strerror.argtypes = [ctypes.c_int]
        L.ardiff_version.restype = ctypes.c_int
        L.ardiff_last_launch_count.restype = ctypes.c_int
        L.ardiff_entropy_gate.restype = ctypes.c_int
        L.ardiff_entropy_gate.argtypes = [vp, i64, i32, f32, vp, vp, vp, vp]
        L.ardiff_entropy_gate_ex.restype = ctypes.c_int
        L.ardiff_entropy_gate_ex.argtypes = [vp, i64, i32, f32, vp, vp, vp, vp, vp]
        L.ardiff_head_create.restype = ctypes.c_int
        L.ardiff_head_create.argtypes = [ctypes.POINTER(HeadDesc), ctypes.POINTER(HeadHostWeights),
                                         ctypes.POINTER(vp)]
        L.ardiff_head_destroy.restype = ctypes.c_int
        L.ardiff_head_destroy.argtypes = [vp]
        L.ardiff_head_sample.restype = ctypes.c_int
        L.ardiff_head_sample.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp]
        L.ardiff_head_status.restype = ctypes.c_int
        L.ardiff_head_status.argtypes = [vp, vp]
        L.ardiff_head_set_timing.restype = ctypes.c_int
        L.ardiff_head_set_timing.argtypes = [vp, ctypes.c_int]
        L.ardiff_head_last_kernel_ms.restype = ctypes.c_int
        L.ardiff_head_last_kernel_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
        L.ardiff_pipeline_create.restype = ctypes.c_int
        L.ardiff_pipeline_create.argtypes = [vp, i64, i32, i32, i32, ctypes.POINTER(vp)]
        L.ardiff_pipeline_destroy.restype = ctypes.c_int
        L.ardiff_pipeline_destroy.argtypes = [vp]
        L.ardiff_pipeline_run_host.restype = ctypes.c_int
        L.ardiff_pipeline_run_host.argtypes = [vp, vp, vp, vp, i64, f32, vp, i32, vp, vp, vp, vp]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().ardiff_strerror(int(code)).decode()


def version() -> int:
    return int(lib().ardiff_version())


def last_launch_count() -> int:
    return int(lib().ardiff_last_launch_count())


def _check(rc: int, where: str):
    if rc != ARDIFF_OK:
        raise ArdiffError(rc, where)


def _stream_ptr(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def ardiff_entropy_gate(feat, tau: float, mask=None, idx=None, count=None, entropy=None,
                        want_entropy: bool = False, stream=None):
    """Entropy gate + compaction on `feat` (torch bf16 CUDA tensor [n, d]).

    Returns (mask u8 [n], idx i32 [n], count i32 [1], entropy f32 [n] or None); outputs are
    allocated here unless passed in. Nothing is synchronised.
    """
    import torch
    assert feat.is_cuda and feat.dtype == torch.bfloat16 and feat.dim() == 2 and feat.is_contiguous()
    n, d = feat.shape
    dev = feat.device
    if mask is None:
        mask = torch.empty((n,), dtype=torch.uint8, device=dev)
    if idx is None:
        idx = torch.empty((max(n, 1),), dtype=torch.int32, device=dev)
    if count is None:
        count = torch.empty((1,), dtype=torch.int32, device=dev)
    if entropy is None and want_entropy:
        entropy = torch.empty((n,), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ardiff_entropy_gate_ex(
            feat.data_ptr(), n, d, float(tau), mask.data_ptr(), idx.data_ptr(), count.data_ptr(),
            entropy.data_ptr() if entropy is not None else None, _stream_ptr(stream))
    _check(rc, "ardiff_entropy_gate")
    return mask, idx, count, entropy


def ardiff_entropy_gate_stats(feat, tau: float = -1.0, want_entropy: bool = False, stream=None):
    """Gate + threshold statistics of its own entropies in one pass. Returns (mask, idx, count, entropy or
    None, out3 float64 CUDA tensor [3] = mean, std, 0.3 mean - 0.1 std)."""
    import torch
    assert feat.is_cuda and feat.dtype == torch.bfloat16 and feat.dim() == 2 and feat.is_contiguous()
    n, d = feat.shape
    dev = feat.device
    mask = torch.empty((n,), dtype=torch.uint8, device=dev)
    idx = torch.empty((max(n, 1),), dtype=torch.int32, device=dev)
    count = torch.empty((1,), dtype=torch.int32, device=dev)
    entropy = torch.empty((n,), dtype=torch.float32, device=dev) if want_entropy else None
    out3 = torch.empty((3,), dtype=torch.float64, device=dev)
    vp = ctypes.c_void_p
    fn = _fn("ardiff_entropy_gate_stats", [vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_float, vp, vp, vp, vp, vp, vp])
    with torch.cuda.device(dev):
        rc = fn(feat.data_ptr(), n, d, float(tau), mask.data_ptr(), idx.data_ptr(), count.data_ptr(),
                entropy.data_ptr() if entropy is not None else None, out3.data_ptr(), _stream_ptr(stream))
    _check(rc, "ardiff_entropy_gate_stats")
    return mask, idx, count, entropy, out3


def _fn(name, argtypes):
    """A library function with its ctypes signature set (lazily, once)."""
    fn = getattr(lib(), name)
    if fn.argtypes is None:
        fn.restype = ctypes.c_int
        fn.argtypes = argtypes
    return fn


def ardiff_entropy_gate_blocks(feat, rows_per_token: int, gamma: int, tau: float, want_token_entropy: bool = False,
                               want_row_entropy: bool = True, stream=None):
    """Block-prefix gate (early stop inside draft blocks of `gamma` tokens, each token owning
    `rows_per_token` rows of feat). Returns (mask u8 [n], idx i32 [n], count i32 [1], block_len i32
    [ceil(n/gamma)], row_entropy f32 [n*rows_per_token], token_entropy f32 [n] or None)."""
    import torch
    assert feat.is_cuda and feat.dtype == torch.bfloat16 and feat.dim() == 2 and feat.is_contiguous()
    rows, d = feat.shape
    assert rows % rows_per_token == 0
    n = rows // rows_per_token
    dev = feat.device
    vp = ctypes.c_void_p
    fn = _fn("ardiff_entropy_gate_blocks", [vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                            ctypes.c_float, vp, vp, vp, vp, vp, vp, vp])
    mask = torch.empty((n,), dtype=torch.uint8, device=dev)
    idx = torch.empty((max(n, 1),), dtype=torch.int32, device=dev)
    count = torch.empty((1,), dtype=torch.int32, device=dev)
    block_len = torch.empty((max((n + gamma - 1) // gamma, 1),), dtype=torch.int32, device=dev)
    row_ent = torch.empty((max(rows, 1),), dtype=torch.float32, device=dev) if want_row_entropy else None
    tok_ent = torch.empty((max(n, 1),), dtype=torch.float32, device=dev) if want_token_entropy else None
    with torch.cuda.device(dev):
        rc = fn(feat.data_ptr(), n, rows_per_token, d, gamma, float(tau),
                row_ent.data_ptr() if row_ent is not None else None,
                tok_ent.data_ptr() if tok_ent is not None else None, mask.data_ptr(), idx.data_ptr(),
                count.data_ptr(), block_len.data_ptr(), _stream_ptr(stream))
    _check(rc, "ardiff_entropy_gate_blocks")
    return mask, idx, count, block_len, row_ent, tok_ent


def ardiff_tau_calibrate(entropy, stream=None):
    """(mean, std, tau = 0.3 mean - 0.1 std) of a float32 CUDA tensor of entropies, as a float64 CUDA tensor [3]."""
    import torch
    assert entropy.is_cuda and entropy.dtype == torch.float32 and entropy.is_contiguous()
    out = torch.empty((3,), dtype=torch.float64, device=entropy.device)
    vp = ctypes.c_void_p
    fn = _fn("ardiff_tau_calibrate", [vp, ctypes.c_int64, vp, vp])
    with torch.cuda.device(entropy.device):
        rc = fn(entropy.data_ptr(), entropy.numel(), out.data_ptr(), _stream_ptr(stream))
    _check(rc, "ardiff_tau_calibrate")
    return out


def ardiff_accept_prefix(r, ratio, gamma: int, block_len=None, stream=None):
    """Accepted draft length per block of `gamma`: first position with r > ratio, else the length of the
    draft (block_len[b] tokens where the early stop truncated block b; the whole block if block_len is None)."""
    import torch
    assert r.is_cuda and r.dtype == torch.float32 and ratio.dtype == torch.float32 and r.shape == ratio.shape
    n = r.numel()
    nb = (n + gamma - 1) // gamma
    out = torch.empty((max(nb, 1),), dtype=torch.int32, device=r.device)
    if block_len is not None:
        assert block_len.is_cuda and block_len.dtype == torch.int32 and block_len.numel() >= nb
    vp = ctypes.c_void_p
    fn = _fn("ardiff_accept_prefix", [vp, vp, ctypes.c_int64, ctypes.c_int32, vp, vp, vp])
    with torch.cuda.device(r.device):
        rc = fn(r.data_ptr(), ratio.data_ptr(), n, gamma, block_len.data_ptr() if block_len is not None else None,
                out.data_ptr(), _stream_ptr(stream))
    _check(rc, "ardiff_accept_prefix")
    return out[:(n + gamma - 1) // gamma]


GATE_NOALLOC_MAX_BLOCKS = 1024
GATE_NOALLOC_MAX_TOKENS = 1 << 24


def ardiff_entropy_gate_noalloc(feat, tau: float, mask, idx, count, stream=None):
    """The gate for callers that may not allocate device memory (a process whose own pool owns the
    device, code inside a stream capture, a latency-critical loop): same kernels and results as
    ardiff_entropy_gate, but the library's scratch is a fixed __device__ array instead of a
    cudaMalloc on first use. Because nothing may be allocated, the caller passes every output
    (mask u8 [n], idx i32 [n], count i32 [1]); there is no entropy output. n is limited to
    GATE_NOALLOC_MAX_TOKENS. Calls on one device share the scratch: do not let two overlap."""
    import torch
    assert feat.is_cuda and feat.dtype == torch.bfloat16 and feat.dim() == 2 and feat.is_contiguous()
    fn = lib().ardiff_entropy_gate_noalloc
    if fn.argtypes is None:
        vp = ctypes.c_void_p
        fn.restype = ctypes.c_int
        fn.argtypes = [vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_float, vp, vp, vp, vp]
    n, d = feat.shape
    with torch.cuda.device(feat.device):
        rc = fn(feat.data_ptr(), n, d, float(tau), mask.data_ptr(), idx.data_ptr(), count.data_ptr(),
                _stream_ptr(stream))
    _check(rc, "ardiff_entropy_gate_noalloc")
    return mask, idx, count


class Head:
    """Owns an ardiff_head handle (device weights + scratch)."""

    def __init__(self, C: int, Dc: int, W: int, L: int, F: int, K_max: int, max_tokens: int,
                 weights: Dict[str, "object"]):
        import numpy as np
        L_ = lib()
        self.desc = HeadDesc(C=C, Dc=Dc, W=W, L=L, F=F, K_max=K_max, max_tokens=max_tokens)
        keep = {k: np.ascontiguousarray(weights[k]) for k in _WEIGHT_FIELDS}
        for k, a in keep.items():
            assert a.dtype == np.uint16, f"{k}: bf16 bit patterns (uint16) expected"
        hw = HeadHostWeights(**{k: keep[k].ctypes.data for k in _WEIGHT_FIELDS})
        h = ctypes.c_void_p()
        _check(L_.ardiff_head_create(ctypes.byref(self.desc), ctypes.byref(hw), ctypes.byref(h)),
               "ardiff_head_create")
        self._h = h

    def ardiff_head_sample(self, cond, noise, t_sched, idx, count, out, stream=None):
        """K = len(t_sched)-1 steps for the survivors idx[0..*count); writes rows of `out`."""
        import numpy as np
        import torch
        assert cond.is_cuda and cond.dtype == torch.bfloat16 and cond.is_contiguous()
        assert noise.is_cuda and noise.dtype == torch.float32 and noise.is_contiguous()
        assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous()
        assert idx.dtype == torch.int32 and count.dtype == torch.int32
        ts = np.ascontiguousarray(t_sched, dtype=np.float32)
        K = ts.shape[0] - 1
        with torch.cuda.device(cond.device):
            rc = lib().ardiff_head_sample(self._h, cond.data_ptr(), noise.data_ptr(), ts.ctypes.data, K,
                                          idx.data_ptr(), count.data_ptr(), out.data_ptr(),
                                          _stream_ptr(stream))
        _check(rc, "ardiff_head_sample")
        return out

    def ardiff_head_sample_coef(self, cond, noise, t_in, coef, idx, count, out, step_noise=None, stream=None):
        """K = len(t_in) head evaluations, each followed by x <- ax x + av v + an z_k.
        coef: [K, 3] (ax, av, an); step_noise: float32 CUDA tensor [K, n, C] or None."""
        import numpy as np
        import torch
        assert cond.is_cuda and cond.dtype == torch.bfloat16 and cond.is_contiguous()
        assert noise.is_cuda and noise.dtype == torch.float32 and noise.is_contiguous()
        assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous()
        ts = np.ascontiguousarray(t_in, dtype=np.float32)
        cf = np.ascontiguousarray(coef, dtype=np.float32)
        K = ts.shape[0]
        assert cf.shape == (K, 3)
        n = noise.shape[0]
        if step_noise is not None:
            assert step_noise.is_cuda and step_noise.dtype == torch.float32 and step_noise.is_contiguous()
            assert tuple(step_noise.shape) == (K, n, noise.shape[1])
        vp = ctypes.c_void_p
        fn = _fn("ardiff_head_sample_coef", [vp, vp, vp, vp, ctypes.c_int32, vp, vp, ctypes.c_int64, vp, vp, vp, vp])
        with torch.cuda.device(cond.device):
            rc = fn(self._h, cond.data_ptr(), noise.data_ptr(), ts.ctypes.data, K, cf.ctypes.data,
                    step_noise.data_ptr() if step_noise is not None else None, n, idx.data_ptr(), count.data_ptr(),
                    out.data_ptr(), _stream_ptr(stream))
        _check(rc, "ardiff_head_sample_coef")
        return out

    def status(self, stream=None) -> int:
        return int(lib().ardiff_head_status(self._h, _stream_ptr(stream)))

    def set_timing(self, on: bool):
        _check(lib().ardiff_head_set_timing(self._h, 1 if on else 0), "ardiff_head_set_timing")

    def last_kernel_ms(self) -> float:
        ms = ctypes.c_float(0.0)
        _check(lib().ardiff_head_last_kernel_ms(self._h, ctypes.byref(ms)), "ardiff_head_last_kernel_ms")
        return float(ms.value)

    def last_kernel_clock_mhz(self, stream=None) -> float:
        """SM clock the last head kernel ran at (cycles / wall time, stamped on the device)."""
        mhz = ctypes.c_double(0.0)
        fn = _fn("ardiff_head_last_kernel_clock", [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_double)])
        _check(fn(self._h, _stream_ptr(stream), ctypes.byref(mhz)), "ardiff_head_last_kernel_clock")
        return float(mhz.value)

    def set_cooperative(self, on: bool):
        fn = _fn("ardiff_head_set_cooperative", [ctypes.c_void_p, ctypes.c_int])
        _check(fn(self._h, 1 if on else 0), "ardiff_head_set_cooperative")

    def inject_stall(self, token_tile: int, wait_limit_us: int):
        """Arms the bounded-wait self-test for the next sample call (see ardiff_head_inject_stall)."""
        fn = _fn("ardiff_head_inject_stall", [ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32])
        _check(fn(self._h, token_tile, wait_limit_us), "ardiff_head_inject_stall")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib().ardiff_head_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Pipeline:
    """Host-buffer front end (ardiff_pipeline_*): device staging for up to max_n tokens.

    With slots >= 2 the overlapped calls (ardiff_pipeline_submit / _wait / _join) are available."""

    def __init__(self, head: Head, max_n: int, d: int, slots: int = 1):
        self.head = head
        self.d, self.Dc, self.C = d, head.desc.Dc, head.desc.C
        self.slots = slots
        self._counts = [ctypes.c_int32(0) for _ in range(slots)]
        p = ctypes.c_void_p()
        vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
        fn = _fn("ardiff_pipeline_create_slots", [vp, i64, i32, i32, i32, i32, ctypes.POINTER(vp)])
        _check(fn(head._h, max_n, d, self.Dc, self.C, slots, ctypes.byref(p)), "ardiff_pipeline_create_slots")
        self._p = p

    def ardiff_pipeline_run_host(self, feat, cond, noise, tau, t_sched, out, mask, stream=None) -> int:
        """feat/cond: host bf16 tensors, noise/out: host f32, mask: host u8 (pinned or not).
        Returns the number of kept tokens. Synchronises the stream."""
        import numpy as np
        ts = np.ascontiguousarray(t_sched, dtype=np.float32)
        n = feat.shape[0]
        count = ctypes.c_int32(0)
        rc = lib().ardiff_pipeline_run_host(self._p, feat.data_ptr(), cond.data_ptr(), noise.data_ptr(), n,
                                            float(tau), ts.ctypes.data, ts.shape[0] - 1, out.data_ptr(),
                                            mask.data_ptr(), ctypes.addressof(count), _stream_ptr(stream))
        _check(rc, "ardiff_pipeline_run_host")
        return int(count.value)

    def ardiff_pipeline_submit(self, slot: int, feat, cond, noise, tau, t_sched, out, mask, stream=None) -> None:
        """Enqueue one batch on `slot` without waiting; the host tensors must stay alive (and should
        be pinned) until ardiff_pipeline_wait(slot)."""
        import numpy as np
        ts = np.ascontiguousarray(t_sched, dtype=np.float32)
        vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float
        fn = _fn("ardiff_pipeline_submit", [vp, i32, vp, vp, vp, i64, f32, vp, i32, vp, vp, vp, vp])
        if not 0 <= slot < self.slots:
            raise ValueError("slot out of range")
        rc = fn(self._p, slot, feat.data_ptr(), cond.data_ptr(), noise.data_ptr(), feat.shape[0], float(tau),
                ts.ctypes.data, ts.shape[0] - 1, out.data_ptr(), mask.data_ptr(),
                ctypes.addressof(self._counts[slot]), _stream_ptr(stream))
        _check(rc, "ardiff_pipeline_submit")

    def ardiff_pipeline_wait(self, slot: int) -> int:
        """Block until the batch on `slot` has been copied out; returns its number of kept tokens."""
        fn = _fn("ardiff_pipeline_wait", [ctypes.c_void_p, ctypes.c_int32])
        _check(fn(self._p, slot), "ardiff_pipeline_wait")
        return int(self._counts[slot].value)

    def ardiff_pipeline_join(self, stream=None) -> None:
        """Make `stream` wait on the device for every batch submitted so far."""
        fn = _fn("ardiff_pipeline_join", [ctypes.c_void_p, ctypes.c_void_p])
        _check(fn(self._p, _stream_ptr(stream)), "ardiff_pipeline_join")

    def close(self):
        if getattr(self, "_p", None) is not None and self._p:
            lib().ardiff_pipeline_destroy(self._p)
            self._p = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
