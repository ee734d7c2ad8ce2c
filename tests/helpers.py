"""Shared helpers of the GPU parity tests: upload, error metrics."""
import numpy as np
import torch

# Tolerances of the parity bar: bf16 outputs max abs <= 2e-2 and mean rel <= 5e-3;
# fp32 outputs max abs error <= 1e-4 of the largest reference magnitude.
BF16_MAX_ABS = 2e-2
BF16_MEAN_REL = 5e-3
F32_REL = 1e-4


def to_device(x: np.ndarray, dtype: str) -> torch.Tensor:
    """float32 numpy (already representable in `dtype`) -> CUDA tensor of that dtype."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def to_host(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def torch_dtype(dtype: str):
    return torch.bfloat16 if dtype == "bf16" else torch.float32


def errors(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    return err.max(), err.mean() / max(np.abs(ref).mean(), 1e-30), err.max() / max(np.abs(ref).max(), 1e-30)


def assert_close(got: np.ndarray, ref: np.ndarray, dtype: str, what: str = ""):
    """max abs = max|g-o|; mean rel = mean|g-o| / mean|o|; fp32 rel = max|g-o| / max|o|."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    max_abs, mean_rel, rel = errors(got, ref)
    if dtype == "bf16":
        assert max_abs <= BF16_MAX_ABS and mean_rel <= BF16_MEAN_REL, \
            f"{what}: max abs {max_abs:.3e} (<= {BF16_MAX_ABS}), mean rel {mean_rel:.3e} (<= {BF16_MEAN_REL})"
    else:
        assert rel <= F32_REL, f"{what}: rel {rel:.3e} (<= {F32_REL})"
