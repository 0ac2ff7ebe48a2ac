"""Shared helpers of the GPU parity tests: numpy inputs -> device tensors, comparisons."""
import numpy as np
import torch


def dev(a, dtype):
    """numpy float32 array (bf16-representable when dtype is bf16) -> CUDA tensor, exact."""
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return t.to(device="cuda", dtype=dtype)


def host64(t):
    return t.detach().to(device="cpu", dtype=torch.float64).numpy()


def check_bf16(got, want, atol=2e-2, rtol=2e-2, what=""):
    """|got - oracle| <= atol + rtol*|oracle| element by element (bf16 configs)."""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want)
    bad = err > atol + rtol * np.abs(want)
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} outside tolerance, max err {err.max():.3e} "
                           f"at {np.unravel_index(err.argmax(), err.shape)}")
    return err.max()


def check_f32(got, want, tol=1e-4, what=""):
    """max |got - oracle| <= tol (fp32 configs)."""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want).max()
    assert err <= tol, f"{what}: max err {err:.3e} > {tol}"
    return err
