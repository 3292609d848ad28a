"""Helpers shared by the GPU parity tests: device upload and the error measure."""
from __future__ import annotations

import numpy as np
import torch

TOL = {"f32": 1e-4, "bf16": 2e-2}     # max relative error per dtype


def dev(a: np.ndarray, dtype: str | None = None) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    if dtype == "bf16":
        t = t.to(torch.bfloat16)          # exact: the values are already bf16-representable
    return t


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def rel_err(got: np.ndarray, want: np.ndarray) -> float:
    """max |got - want| / max(|want|, rms of want's row): near-zero elements are measured
    against the size of their row instead of against themselves."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    rms = np.sqrt(np.mean(want * want, axis=-1, keepdims=True))
    den = np.maximum(np.abs(want), np.maximum(rms, 1e-30))
    return float(np.max(np.abs(got - want) / den))


def weights_to_device(wts: dict, dtype: str) -> dict:
    return {k: dev(v, dtype) for k, v in wts.items()}
