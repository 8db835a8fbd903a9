"""Shared helpers of the GPU parity tests: tolerances and comparison against the fp64 oracle."""
import numpy as np
import torch

# bf16 operands, fp32 accumulation, bf16 output: the bounds the library is held to.
O_MAX_ABS = 2e-2
O_MEAN_ABS = 2e-3
LSE_MAX_ABS = 1e-3


def gpu_available() -> bool:
    return torch.cuda.is_available()


def compare(o_gpu: torch.Tensor, lse_gpu: torch.Tensor, o_ref: np.ndarray, lse_ref: np.ndarray, what=""):
    """Element-by-element comparison; returns the error statistics after asserting the bounds."""
    o = o_gpu.detach().double().cpu().numpy()
    lse = lse_gpu.detach().double().cpu().numpy()
    assert o.shape == o_ref.shape, (o.shape, o_ref.shape)
    assert lse.shape == lse_ref.shape, (lse.shape, lse_ref.shape)
    assert np.isfinite(o).all() and np.isfinite(lse).all(), f"{what}: non-finite output"
    err = np.abs(o - o_ref)
    lerr = np.abs(lse - lse_ref)
    stats = dict(o_max=float(err.max()), o_mean=float(err.mean()), lse_max=float(lerr.max()),
                 argmax=tuple(int(x) for x in np.unravel_index(err.argmax(), err.shape)))
    assert stats["o_max"] <= O_MAX_ABS, f"{what}: O max-abs {stats}"
    assert stats["o_mean"] <= O_MEAN_ABS, f"{what}: O mean-abs {stats}"
    assert stats["lse_max"] <= LSE_MAX_ABS, f"{what}: LSE max-abs {stats}"
    return stats
