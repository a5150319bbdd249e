"""Helpers shared by the GPU parity tests: numpy <-> torch marshalling and the acceptance rule."""
import numpy as np


def to_bf16_cuda(bits):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_to_f64(t):
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def bits_of(t):
    """Raw little-endian bytes of a torch tensor as a numpy uint8 array (bit-exact comparisons)."""
    import torch
    return t.detach().contiguous().view(torch.uint8).cpu().numpy().reshape(-1)


def cuda(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


# Acceptance rule for bf16 outputs: per output row m, max_n |y - y_ref| <= 1e-2 * max_n |y_ref[m][:]|.
# The arithmetic supports a tighter figure, which the tests assert: bf16 keeps 8 significant bits, so
# the final rounding costs at most half an ulp = 2^-8 of |y| (<= 2^-8 of the row maximum), and fp32
# accumulation over K <= 11008 terms plus the 128-offset cancellation stay under 2^-11 of the row maximum.
CONTRACT_REL = 1e-2
DERIVED_REL = 2.0 ** -8 + 2.0 ** -11


def assert_rows_close(y, y_ref, rel=DERIVED_REL):
    y = np.asarray(y, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    assert y.shape == y_ref.shape
    assert np.all(np.isfinite(y))
    tol = rel * np.abs(y_ref).max(axis=1, keepdims=True)
    err = np.abs(y - y_ref)
    worst = (err / np.maximum(tol, 1e-300)).max() if y.size else 0.0
    assert np.all(err <= tol + 1e-30), f"row-relative error {worst * rel:.3e} exceeds {rel:.1e}"
