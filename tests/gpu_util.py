"""Helpers shared by the GPU parity tests: contexts, padded device tensors, exact comparison."""
import numpy as np
import torch

from paper_2207_01405_b200 import binding, build

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        build.build()
        _ctx = binding.Context(0)
    return _ctx


def dev(a: np.ndarray, pad_to: int = 16) -> torch.Tensor:
    """Uploads a 2-D / 3-D array with its last dimension padded (stride multiple of pad_to); returns the unpadded view."""
    a = np.ascontiguousarray(a)
    n = a.shape[-1]
    ld = (n + pad_to - 1) // pad_to * pad_to
    buf = torch.zeros(a.shape[:-1] + (ld,), dtype=torch.from_numpy(a[..., :0].copy()).dtype, device="cuda")
    buf[..., :n] = torch.from_numpy(a).cuda()
    return buf[..., :n]


def host(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy()


def assert_equal(got: np.ndarray, want: np.ndarray, what: str = ""):
    """Bit-exact comparison with a first-mismatch report."""
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if not np.array_equal(got, want):
        bad = np.argwhere(got != want)
        i = tuple(bad[0])
        raise AssertionError(f"{what}: {len(bad)} mismatches of {got.size}; first at {i}: got {got[i]} want {want[i]}")
