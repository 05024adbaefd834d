"""Seeded synthetic inputs and the workload table shared by the tests and the benchmark.

This package holds none of the method's arithmetic. It draws the feature, conditioning,
noise and weight arrays (counter-based generator in ``gen.c``; any row range can be
produced on its own) and names the five workload shapes. Both the CPU oracle's callers
and the CUDA path's callers take their inputs from here, so the two see identical bits.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "_gen.so")
_lib = None

KIND_FLAT, KIND_PEAKED, KIND_HEAVY = 0, 1, 2

# stream ids (each array has its own stream; features use 3 consecutive ids)
_S_FEAT, _S_COND, _S_NOISE, _S_WEIGHT0 = 10, 20, 30, 100


def build(force: bool = False) -> str:
    """Compile gen.c into _gen.so (gcc, OpenMP). Returns the library path."""
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
        u64, i64, i32, dbl, vp = (ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32,
                                  ctypes.c_double, ctypes.c_void_p)
        lib.synth_normal_f32.argtypes = [u64, u64, u64, u64, dbl, vp]
        lib.synth_normal_bf16.argtypes = [u64, u64, u64, u64, dbl, vp]
        lib.synth_feat_rows.argtypes = [u64, u64, i32, dbl, i32, i32, i64, i64, i32, vp, vp]
        lib.synth_bf16_to_f32.argtypes = [vp, u64, vp]
        lib.synth_f32_to_bf16.argtypes = [vp, u64, vp]
        for f in (lib.synth_normal_f32, lib.synth_normal_bf16, lib.synth_feat_rows,
                  lib.synth_bf16_to_f32, lib.synth_f32_to_bf16):
            f.restype = None
        _lib = lib
    return _lib


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float32, exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float32)
    _load().synth_bf16_to_f32(_ptr(bits), bits.size, _ptr(out))
    return out


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 bit patterns (uint16), nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().synth_f32_to_bf16(_ptr(x), x.size, _ptr(out))
    return out


@dataclass(frozen=True)
class Workload:
    """Shapes and input recipe of one synthetic workload."""
    name: str
    n: int            # draft tokens
    d: int            # shallow-feature channels per token (gate input width)
    C: int            # token (latent) dim
    Dc: int           # conditioning (AR hidden state) dim
    W: int            # head width
    L: int            # AdaLN residual blocks
    K: int            # sampler steps
    seed: int
    feat_mode: int    # 0 alternate kinds by row parity, 1 Bernoulli(p_a)
    p_a: float
    kind_a: int
    kind_b: int
    filter_q: float   # fraction of tokens the gate should drop (tau = that quantile)
    F: int = 256      # time-embedding frequencies (cos half + sin half)

    def flops_per_token(self, K: Optional[int] = None) -> float:
        K = self.K if K is None else K
        W, C = self.W, self.C
        return 2.0 * self.Dc * W + K * (self.L * 10.0 * W * W + 4.0 * W * W + 4.0 * C * W)

    def gate_bytes(self) -> float:
        return self.n * (2.0 * self.d + 5.0) + 4.0


def _seed(cfg: int) -> int:
    return 20251208 * 10 + cfg


WORKLOADS: Dict[str, Workload] = {
    "cfg1": Workload("cfg1", 64, 256, 16, 256, 256, 2, 4, _seed(1), 0, 0.5, KIND_FLAT, KIND_PEAKED, 0.5),
    "cfg2": Workload("cfg2", 64 * 256, 768, 16, 768, 1024, 3, 4, _seed(2), 1, 0.3, KIND_PEAKED, KIND_FLAT, 0.3),
    "cfg3": Workload("cfg3", 256 * 256, 1024, 16, 1024, 1536, 6, 4, _seed(3), 1, 0.4, KIND_PEAKED, KIND_FLAT, 0.4),
    "cfg4": Workload("cfg4", 32 * 1024, 5120, 64, 5120, 1536, 12, 4, _seed(4), 1, 0.7, KIND_HEAVY, KIND_PEAKED, 0.3),
    # gate stress: features as cfg4, head as cfg2 (its cond is a separate [n x 768] array)
    "cfg5": Workload("cfg5", 1 << 20, 5120, 16, 768, 1024, 3, 4, _seed(5), 1, 0.7, KIND_HEAVY, KIND_PEAKED, 0.5),
}


def workload(name: str, **overrides) -> Workload:
    wl = WORKLOADS[name]
    return replace(wl, **overrides) if overrides else wl


def features(wl: Workload, row0: int = 0, nrows: Optional[int] = None, return_kinds: bool = False):
    """bf16 bits [nrows, d] of feature rows row0 .. row0+nrows-1."""
    nrows = wl.n - row0 if nrows is None else nrows
    out = np.empty((nrows, wl.d), dtype=np.uint16)
    kinds = np.empty((nrows,), dtype=np.uint8)
    _load().synth_feat_rows(wl.seed, _S_FEAT, wl.feat_mode, wl.p_a, wl.kind_a, wl.kind_b,
                            row0, nrows, wl.d, _ptr(out), _ptr(kinds))
    return (out, kinds) if return_kinds else out


def cond(wl: Workload, row0: int = 0, nrows: Optional[int] = None) -> np.ndarray:
    """bf16 bits [nrows, Dc]: the AR hidden state of each token, N(0,1)."""
    nrows = wl.n - row0 if nrows is None else nrows
    out = np.empty((nrows, wl.Dc), dtype=np.uint16)
    _load().synth_normal_bf16(wl.seed, _S_COND, row0 * wl.Dc, nrows * wl.Dc, 1.0, _ptr(out))
    return out


def noise(wl: Workload, row0: int = 0, nrows: Optional[int] = None) -> np.ndarray:
    """float32 [nrows, C]: the start noise of each token, N(0,1)."""
    nrows = wl.n - row0 if nrows is None else nrows
    out = np.empty((nrows, wl.C), dtype=np.float32)
    _load().synth_normal_f32(wl.seed, _S_NOISE, row0 * wl.C, nrows * wl.C, 1.0, _ptr(out))
    return out


def t_sched(K: int) -> np.ndarray:
    """float32 [K+1]: t_k = k/K (noise at t=0, sample at t=1)."""
    if K == 0:
        return np.zeros((1,), dtype=np.float32)
    return (np.arange(K + 1, dtype=np.float64) / K).astype(np.float32)


# name -> (shape function, fan_in function); Linear layout [out, in], biases [out]
def weight_shapes(wl: Workload):
    C, Dc, W, L, F = wl.C, wl.Dc, wl.W, wl.L, wl.F
    return {
        "Wc": ((W, Dc), Dc), "bc": ((W,), Dc),
        "Wt1": ((W, F), F), "bt1": ((W,), F),
        "Wt2": ((W, W), W), "bt2": ((W,), W),
        "Win": ((W, C), C), "bin": ((W,), C),
        "Wmod": ((L, 3 * W, W), W), "bmod": ((L, 3 * W), W),
        "W1": ((L, W, W), W), "b1": ((L, W), W),
        "W2": ((L, W, W), W), "b2": ((L, W), W),
        "Wfm": ((2 * W, W), W), "bfm": ((2 * W,), W),
        "Wout": ((C, W), W), "bout": ((C,), W),
    }


def head_weights(wl: Workload, std: Optional[float] = 0.02) -> Dict[str, np.ndarray]:
    """All head parameters as bf16 bits. std=None draws each tensor with 1/sqrt(fan_in)."""
    out = {}
    for k, (name, (shape, fan_in)) in enumerate(weight_shapes(wl).items()):
        a = np.empty(shape, dtype=np.uint16)
        s = std if std is not None else 1.0 / float(np.sqrt(fan_in))
        _load().synth_normal_bf16(wl.seed, _S_WEIGHT0 + k, 0, a.size, s, _ptr(a))
        out[name] = a
    return out
