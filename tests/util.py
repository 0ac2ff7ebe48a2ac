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


class Guarded:
    """A device tensor placed inside a larger sentinel-filled allocation (compute-sanitizer stand-in).

    `t` is the tensor to hand to the library: `shape` elements of `dtype`, rows `pitch` elements apart
    (default: dense), starting 256-byte aligned.  Every byte of the allocation that does not belong to an
    element of `t` - a band before it, a band after it, and the gap at the end of every row when
    pitch > shape[-1] - is filled with SENTINEL.  check() asserts that all of them still hold it, i.e.
    that no kernel stored outside the tensor."""
    SENTINEL = 0xA5
    BAND = 8192

    def __init__(self, shape, dtype, pitch=None, fill=None):
        shape = tuple(int(s) for s in shape)
        item = torch.empty((), dtype=dtype).element_size()
        cols = shape[-1] if shape else 1
        rows = 1
        for s in shape[:-1]:
            rows *= s
        self.pitch = cols if pitch is None else int(pitch)
        assert self.pitch >= cols
        self.rows, self.cols, self.item = rows, cols, item
        self.nbytes = rows * self.pitch * item
        self.buf = torch.full((self.BAND + self.nbytes + self.BAND,), self.SENTINEL, dtype=torch.uint8, device="cuda")
        assert self.buf.data_ptr() % 256 == 0
        body = self.buf[self.BAND:self.BAND + self.nbytes].view(dtype)
        if self.pitch == cols:
            self.t = body.view(shape)
        else:
            assert len(shape) == 2
            self.t = body.view(rows, self.pitch)[:, :cols]
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what=""):
        torch.cuda.synchronize()
        s = self.SENTINEL
        assert bool((self.buf[:self.BAND] == s).all()), f"{what}: a store landed BEFORE the tensor"
        assert bool((self.buf[self.BAND + self.nbytes:] == s).all()), f"{what}: a store landed PAST the tensor's end"
        if self.pitch != self.cols and self.rows > 0:
            gaps = self.buf[self.BAND:self.BAND + self.nbytes].view(self.rows, self.pitch * self.item)[:, self.cols * self.item:]
            assert bool((gaps == s).all()), f"{what}: a store landed in the gap between two rows"


def guarded_workspace(nbytes):
    """A workspace of exactly `nbytes` bytes between two sentinel bands; returns (Guarded, uint8 tensor)."""
    g = Guarded((max(int(nbytes), 0),), torch.uint8)
    return g, g.t


def ints(rng, shape, lo=-3, hi=3):
    """Small-integer test operands as float32: products and sums of a few thousand of them are exact in
    fp32 (and in the oracle's fp64), so GPU and oracle must agree bit for bit."""
    return rng.integers(lo, hi + 1, shape).astype(np.float32)
