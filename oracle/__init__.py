"""ORACLE -- test infrastructure, not product code.

ctypes front end of ``ardiff_oracle.c``: the slow fp64 CPU statement of the entropy gate
(softmax-row entropy, threshold, ascending survivor list; the paper's entropy indicator
and Algorithm 1's "H^s < tau_ent" test) and of the K-step AdaLN residual-MLP flow head.
Only tests, the smoke check and the benchmark's cpu_baseline / reference leg may import
this package. It imports nothing from the CUDA package.

The head's architecture details are this build's reading of "MLP-based head conditioned
on t and z" (parity unpinned with respect to the paper for those details); the CPU tests
pin the functions to closed forms, invariants, library routines and brute force.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ardiff_oracle.c")
_LIB = os.path.join(_HERE, "_oracle.so")
_lib = None

_PARAM_ORDER = ["Wc", "bc", "Wt1", "bt1", "Wt2", "bt2", "Win", "bin", "Wmod", "bmod",
                "W1", "b1", "W2", "b2", "Wfm", "bfm", "Wout", "bout"]


class _HeadParams(ctypes.Structure):
    _fields_ = ([(k, ctypes.c_int32) for k in ("C", "Dc", "W", "L", "F")]
                + [(k, ctypes.c_void_p) for k in _PARAM_ORDER])


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O2, OpenMP, no fast-math). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
        lib.oracle_entropy.argtypes = [vp, i64, i32, vp]
        lib.oracle_gate.argtypes = [vp, i64, i32, ctypes.c_float, vp, vp, vp, vp]
        lib.oracle_head_sample.argtypes = [ctypes.POINTER(_HeadParams), vp, vp, vp, i32, vp, i32, vp]
        lib.oracle_head_sample_coef.argtypes = [ctypes.POINTER(_HeadParams), vp, vp, vp, i32, vp, vp, i64, vp, i32, vp]
        lib.oracle_gate_blocks.argtypes = [vp, i64, i32, i32, i32, ctypes.c_float, vp, vp, vp, vp, vp]
        lib.oracle_tau_calibrate.argtypes = [vp, i64, vp, vp, vp]
        lib.oracle_accept_prefix.argtypes = [vp, vp, i64, i32, vp, vp]
        lib.oracle_layer_norm.argtypes = [vp, i32, vp]
        lib.oracle_time_embedding.argtypes = [ctypes.POINTER(_HeadParams), ctypes.c_float, vp]
        for f in (lib.oracle_entropy, lib.oracle_gate, lib.oracle_head_sample, lib.oracle_head_sample_coef,
                  lib.oracle_gate_blocks, lib.oracle_tau_calibrate, lib.oracle_accept_prefix,
                  lib.oracle_layer_norm, lib.oracle_time_embedding):
            f.restype = None
        _lib = lib
    return _lib


def threads() -> int:
    """OpenMP threads the oracle will use (OMP_NUM_THREADS, else the cores this process may run on)."""
    v = os.environ.get("OMP_NUM_THREADS")
    if v:
        return int(v.split(",")[0])
    return len(os.sched_getaffinity(0))


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 arrays are passed as uint16 bit patterns"
    return a


def entropy(feat_bits: np.ndarray) -> np.ndarray:
    """H[i] = -sum_c softmax(feat[i])_c ln softmax(feat[i])_c, fp64. feat: uint16 bf16 bits [n, d]."""
    feat_bits = _u16(feat_bits)
    n, d = feat_bits.shape
    H = np.empty((n,), dtype=np.float64)
    _load().oracle_entropy(feat_bits.ctypes.data, n, d, H.ctypes.data)
    return H


def gate(feat_bits: np.ndarray, tau: float) -> Tuple[np.ndarray, np.ndarray, np.ndarray, int]:
    """(H [n] f64, mask [n] u8, idx [count] i32 ascending, count). keep iff H >= float32(tau)."""
    feat_bits = _u16(feat_bits)
    n, d = feat_bits.shape
    H = np.empty((n,), dtype=np.float64)
    mask = np.empty((n,), dtype=np.uint8)
    idx = np.empty((max(n, 1),), dtype=np.int32)
    count = ctypes.c_int32(0)
    _load().oracle_gate(feat_bits.ctypes.data, n, d, ctypes.c_float(np.float32(tau)),
                        H.ctypes.data, mask.ctypes.data, idx.ctypes.data, ctypes.byref(count))
    return H, mask, idx[:count.value].copy(), int(count.value)


def _params(weights: Dict[str, np.ndarray], F: Optional[int] = None):
    keep = {k: _u16(weights[k]) for k in _PARAM_ORDER}
    W, Dc = keep["Wc"].shape
    C = keep["Wout"].shape[0]
    L = keep["Wmod"].shape[0]
    Fdim = keep["Wt1"].shape[1]
    assert F is None or F == Fdim
    assert keep["Wmod"].shape == (L, 3 * W, W) and keep["Wfm"].shape == (2 * W, W)
    assert keep["Win"].shape == (W, C) and keep["W1"].shape == (L, W, W)
    p = _HeadParams(C=C, Dc=Dc, W=W, L=L, F=Fdim, **{k: keep[k].ctypes.data for k in _PARAM_ORDER})
    return p, keep


def head_sample(weights: Dict[str, np.ndarray], cond_bits: np.ndarray, noise: np.ndarray,
                t_sched: np.ndarray, idx: np.ndarray, out: Optional[np.ndarray] = None) -> np.ndarray:
    """K = len(t_sched)-1 Euler flow steps of the head for the tokens in idx.

    Returns out [n, C] float64; rows not named in idx are left as they were (zeros if out is None).
    """
    p, keep = _params(weights)
    cond_bits = _u16(cond_bits)
    noise = np.ascontiguousarray(noise, dtype=np.float32)
    t_sched = np.ascontiguousarray(t_sched, dtype=np.float32)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    n = noise.shape[0]
    assert cond_bits.shape == (n, p.Dc) and noise.shape == (n, p.C)
    K = t_sched.shape[0] - 1
    assert K >= 0
    if out is None:
        out = np.zeros((n, p.C), dtype=np.float64)
    assert out.dtype == np.float64 and out.flags["C_CONTIGUOUS"] and out.shape == (n, p.C)
    _load().oracle_head_sample(ctypes.byref(p), cond_bits.ctypes.data, noise.ctypes.data,
                               t_sched.ctypes.data, K, idx.ctypes.data, idx.shape[0], out.ctypes.data)
    del keep
    return out


def head_sample_coef(weights: Dict[str, np.ndarray], cond_bits: np.ndarray, noise: np.ndarray,
                     t_in: np.ndarray, coef: np.ndarray, idx: np.ndarray,
                     step_noise: Optional[np.ndarray] = None) -> np.ndarray:
    """K = len(t_in) head evaluations at times t_in, each followed by x <- ax x + av v + an z_k.

    coef: float32 [K, 3] = (ax, av, an) per step; step_noise: float32 [K, n, C] or None.
    Returns out [n, C] float64 (rows not in idx are zero)."""
    p, keep = _params(weights)
    cond_bits = _u16(cond_bits)
    noise = np.ascontiguousarray(noise, dtype=np.float32)
    t_in = np.ascontiguousarray(t_in, dtype=np.float32)
    coef = np.ascontiguousarray(coef, dtype=np.float32)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    n = noise.shape[0]
    K = t_in.shape[0]
    assert coef.shape == (K, 3)
    sn = None
    if step_noise is not None:
        sn = np.ascontiguousarray(step_noise, dtype=np.float32)
        assert sn.shape == (K, n, p.C)
    out = np.zeros((n, p.C), dtype=np.float64)
    _load().oracle_head_sample_coef(ctypes.byref(p), cond_bits.ctypes.data, noise.ctypes.data, t_in.ctypes.data, K,
                                    coef.ctypes.data, sn.ctypes.data if sn is not None else None, n,
                                    idx.ctypes.data, idx.shape[0], out.ctypes.data)
    del keep
    return out


def gate_blocks(feat_bits: np.ndarray, rows_per_token: int, gamma: int, tau: float):
    """Block-prefix gate (Algorithm 1, Step 1). feat: bf16 bits [n * rows_per_token, d].

    Returns (Hs [n] f64 token indicators, mask [n] u8, idx [count] i32, count, len [ceil(n/gamma)] i32)."""
    feat_bits = _u16(feat_bits)
    rows, d = feat_bits.shape
    assert rows % rows_per_token == 0 and gamma >= 1
    n = rows // rows_per_token
    nb = (n + gamma - 1) // gamma
    Hs = np.empty((n,), dtype=np.float64)
    mask = np.empty((n,), dtype=np.uint8)
    idx = np.empty((max(n, 1),), dtype=np.int32)
    ln = np.empty((max(nb, 1),), dtype=np.int32)
    count = ctypes.c_int32(0)
    _load().oracle_gate_blocks(feat_bits.ctypes.data, n, rows_per_token, d, gamma, ctypes.c_float(np.float32(tau)),
                               Hs.ctypes.data, mask.ctypes.data, idx.ctypes.data, ctypes.byref(count), ln.ctypes.data)
    return Hs, mask, idx[:count.value].copy(), int(count.value), ln[:nb].copy()


def tau_calibrate(H: np.ndarray) -> Tuple[float, float, float]:
    """(mean, std, tau = 0.3 mean - 0.1 std) of a set of entropies (std with divisor n)."""
    H = np.ascontiguousarray(H, dtype=np.float64)
    m, s, t = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    _load().oracle_tau_calibrate(H.ctypes.data, H.shape[0], ctypes.byref(m), ctypes.byref(s), ctypes.byref(t))
    return m.value, s.value, t.value


def accept_prefix(r: np.ndarray, ratio: np.ndarray, gamma: int, block_len: Optional[np.ndarray] = None) -> np.ndarray:
    """Accepted draft length per block of gamma: first position whose r exceeds its ratio, else the length of
    the draft (block_len[b] where the early stop truncated the block, the whole block otherwise)."""
    r = np.ascontiguousarray(r, dtype=np.float32)
    ratio = np.ascontiguousarray(ratio, dtype=np.float32)
    n = r.shape[0]
    nb = (n + gamma - 1) // gamma
    out = np.empty((max(nb, 1),), dtype=np.int32)
    bl = None
    if block_len is not None:
        bl = np.ascontiguousarray(block_len, dtype=np.int32)
        assert bl.shape == (nb,)
    _load().oracle_accept_prefix(r.ctypes.data, ratio.ctypes.data, n, gamma,
                                 bl.ctypes.data if bl is not None else None, out.ctypes.data)
    return out[:nb].copy()


def layer_norm(h: np.ndarray) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.float64)
    out = np.empty_like(h)
    _load().oracle_layer_norm(h.ctypes.data, h.shape[0], out.ctypes.data)
    return out


def time_embedding(weights: Dict[str, np.ndarray], t: float) -> np.ndarray:
    p, keep = _params(weights)
    out = np.empty((p.W,), dtype=np.float64)
    _load().oracle_time_embedding(ctypes.byref(p), ctypes.c_float(np.float32(t)), out.ctypes.data)
    del keep
    return out
