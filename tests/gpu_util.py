"""Helpers shared by the GPU parity tests: tolerances and tensor transfer."""
import numpy as np
import torch


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def assert_rows_close(got: np.ndarray, ref: np.ndarray, rel: float = 1e-5, what: str = ""):
    """fp32 aggregation tolerance: per row, max |gpu - ref| <= rel * ||ref row||_2,
    and exactly 0 where the reference row is exactly 0."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    ref64, got64 = ref.astype(np.float64), got.astype(np.float64)
    norm = np.linalg.norm(ref64, axis=1)
    err = np.abs(got64 - ref64).max(axis=1) if ref.shape[1] else np.zeros(ref.shape[0])
    zero = norm == 0
    assert np.all(got64[zero] == 0), what + ": rows that must be exactly zero are not"
    bad = err > rel * norm
    assert not bad.any(), "%s: %d rows out of tolerance, worst err/norm = %.3g" % (
        what, int(bad.sum()), float((err[~zero] / norm[~zero]).max()))


def assert_logits_close(got: np.ndarray, ref: np.ndarray, rel: float = 2e-2, what: str = ""):
    """bf16-operand MLP tolerance: |gpu - ref| <= rel * scale, where the scale of a row is its
    largest |logit|, but not less than the RMS logit of the whole batch (a row whose logits all
    happen to be near zero is judged against the size logits have in this model)."""
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    scale = np.maximum(np.abs(ref).max(axis=1, keepdims=True), max(rms, 1e-6))
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64)) / scale
    assert err.max() <= rel, "%s: worst relative logit error %.3g > %.3g" % (what, float(err.max()), rel)
