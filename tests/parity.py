"""Comparison helpers for CUDA-vs-oracle parity tests.

Protocol: integer outputs must be bit-exact, except elements whose deciding
score gap is below 1e-3 relative (the oracle reports that near-tie set);
mismatches are counted and must lie inside the set.  Scores: max abs error
relative to the largest |score| of the segment.  Feature rows: relative L2
error, compared on rows whose member sets agree.  Gathers: bit-exact.
"""

from __future__ import annotations

import numpy as np
import torch

TOL = {"bf16": 2e-2, "f32": 1e-5}


def to_torch(x: np.ndarray, dtype: str, device="cuda") -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)          # exact: values are bf16-representable
    return t.to(device)


def to_np(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy().astype(np.float64)
    return t.cpu().numpy()


def bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit patterns, for bit-exact comparisons."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    if t.dtype == torch.float32:
        return t.view(torch.int32).cpu().numpy().view(np.uint32)
    return t.cpu().numpy()


def score_err(got: np.ndarray, want: np.ndarray) -> float:
    scale = max(float(np.max(np.abs(want))), 1e-300)
    return float(np.max(np.abs(got.astype(np.float64) - want))) / scale


def check_scores(got, want, dtype, what=""):
    err = score_err(np.asarray(got), np.asarray(want))
    assert err <= TOL[dtype], f"{what}: relative score error {err:.3e} > {TOL[dtype]}"
    return err


def check_index_set(got_idx, want_idx, near_mask_by_index, what=""):
    """Both are index lists; every index in the symmetric difference must be a near-tie."""
    g, w = set(int(i) for i in got_idx), set(int(i) for i in want_idx)
    diff = sorted(g ^ w)
    bad = [i for i in diff if not near_mask_by_index(i)]
    assert not bad, f"{what}: {len(bad)} mismatches outside the near-tie band, e.g. {bad[:8]}"
    return len(diff)


def row_rel_l2(got: np.ndarray, want: np.ndarray) -> np.ndarray:
    num = np.sqrt(np.sum((got.astype(np.float64) - want) ** 2, axis=1))
    den = np.maximum(np.sqrt(np.sum(want ** 2, axis=1)), 1e-300)
    return num / den
