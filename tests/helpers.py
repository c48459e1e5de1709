"""Shared checks for the GPU parity tests."""
import numpy as np
import torch

ABS_TOL = 2e-2
REL_TOL = 2e-2


def check_against_oracle(got_bf16: torch.Tensor, ref: np.ndarray, what: str = ""):
    """GPU bf16 output (converted exactly to float64) against the unrounded float64 oracle.

    Passes iff every element has |err| <= 2e-2 AND |err| <= 2e-2 * max(|ref|, rms of its row): the
    relative error is floored at the row's RMS so that near-zero elements of a cancelling sum are not
    divided by ~0.  Returns (max abs err, max floored-relative err) for reporting.
    """
    got = got_bf16.detach().to("cpu").to(torch.float64).numpy()
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    rms = np.sqrt((ref ** 2).mean(axis=-1, keepdims=True))
    floor = np.maximum(np.abs(ref), rms)
    rel = err / np.maximum(floor, 1e-30)
    max_abs, max_rel = float(err.max(initial=0.0)), float(rel.max(initial=0.0))
    assert max_abs <= ABS_TOL, f"{what}: max abs err {max_abs:.4g} > {ABS_TOL}"
    assert max_rel <= REL_TOL, f"{what}: max rel err {max_rel:.4g} > {REL_TOL}"
    return max_abs, max_rel
