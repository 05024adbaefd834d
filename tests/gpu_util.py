"""Helpers for the GPU parity tests (device upload of synthetic arrays)."""
import numpy as np
import torch


def require_cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device (run them with -m gpu on a B200)"
    return torch.device("cuda:0")


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 CUDA tensor of the same shape."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(require_cuda())
    return t.view(torch.bfloat16)


def dev_f32(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(require_cuda())


HEAD_REL_TOL = 2e-2


def assert_head_parity(got, want, rows, what="out", model=None):
    """Per token: max |got - oracle| <= 2e-2 x RMS(oracle row).

    With bf16 operands a few tokens of the deepest single-step workloads sit at that bar by rounding alone
    (tests/test_rounding_model.py). `model(rows) -> error ratios of the CPU rounding model` is consulted only
    for rows that miss the bar: such a row passes if rounding alone already costs it more than half of the
    bar and the kernel stays within twice that floor; at most 1 % of the rows (never more than 4) may need
    this. Anything else is a kernel error."""
    rows = np.asarray(rows)
    err = np.abs(got[rows].astype(np.float64) - want[rows]).max(axis=1)
    rms = np.sqrt((want[rows] ** 2).mean(axis=1))
    ratio = err / rms
    bad = np.flatnonzero(ratio > HEAD_REL_TOL)
    if len(bad) == 0:
        return float(ratio.max())
    assert model is not None, f"{what}: worst max|err|/rms = {ratio.max():.3e}"
    assert len(bad) <= min(4, max(1, len(rows) // 100)), f"{what}: {len(bad)} of {len(rows)} rows beyond {HEAD_REL_TOL}"
    floor = np.asarray(model(rows[bad]))
    for b, f in zip(bad, floor):
        assert f > 0.5 * HEAD_REL_TOL and ratio[b] <= 2.0 * f, \
            f"{what}: row {rows[b]} at {ratio[b]:.3e}, bf16 rounding alone gives {f:.3e}"
    return float(ratio.max())
