"""Helpers for the GPU-vs-oracle parity tests (comparison rules only; no method arithmetic)."""
import numpy as np
import torch

SCORE_RTOL = 2e-3      # max relative error of pooled scores (bf16 inputs, fp32 accumulation)
SCORE_FLOOR = 1e-12    # |ref| floor of the relative error (scores of a unit add up to ~M)
BAND = 4e-3            # index sets may differ only where the oracle score is within BAND of theta


def score_rel_err(gpu_scores: np.ndarray, ref_scores: np.ndarray) -> float:
    ref = np.asarray(ref_scores, np.float64)
    got = np.asarray(gpu_scores, np.float64)
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), SCORE_FLOOR)))


def check_index_set(idx_gpu: np.ndarray, idx_ref: np.ndarray, ref_scores: np.ndarray, L: int,
                    R: int, B: int) -> int:
    """Checks one unit's kept positions. What is unique must match: B entries, the first B-R
    strictly ascending in [0, L-R), the tail last, and the same set as the oracle except at
    positions whose oracle score ties with the B-R-th largest within BAND. Returns the number of
    positions that differ (all inside the band)."""
    Kb, Ls = B - R, L - R
    idx_gpu = np.asarray(idx_gpu)
    assert idx_gpu.shape == (B,)
    head = idx_gpu[:Kb]
    assert (head >= 0).all() and (head < Ls).all()
    assert (np.diff(head) > 0).all()
    assert idx_gpu[Kb:].tolist() == list(range(Ls, L))
    got, want = set(head.tolist()), set(np.asarray(idx_ref)[:Kb].tolist())
    if got == want:
        return 0
    theta = np.sort(ref_scores)[::-1][Kb - 1]
    diff = np.array(sorted(got ^ want))
    off = np.abs(ref_scores[diff] - theta)
    assert (off <= BAND * theta).all(), (
        f"{len(diff)} positions differ outside the tie band: worst {off.max() / theta:.3e}")
    return len(diff)


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
