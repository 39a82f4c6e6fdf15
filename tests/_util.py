"""Helpers shared by the GPU parity tests: tensor marshalling and the parity bar."""
import numpy as np
import torch

REL_L2 = 1e-3          # relative L2 error per tensor
MAX_ABS = 1e-2         # max abs error, as a fraction of max |reference|


def dev_bf16(a: np.ndarray) -> torch.Tensor:
    """numpy float array holding bf16-representable values -> cuda bfloat16 tensor (exact)."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().to(torch.bfloat16)


def host_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def assert_close(got: np.ndarray, ref: np.ndarray, what: str, rel=REL_L2, mx=MAX_ABS):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    nr = np.linalg.norm(ref)
    err = np.linalg.norm(got - ref)
    mabs = np.abs(got - ref).max() if got.size else 0.0
    mref = np.abs(ref).max() if ref.size else 0.0
    assert err <= rel * nr + 1e-30, f"{what}: rel L2 {err / max(nr, 1e-300):.3e} > {rel}"
    assert mabs <= mx * mref + 1e-30, f"{what}: max abs {mabs:.3e} > {mx} * {mref:.3e}"
    return err / max(nr, 1e-300)
