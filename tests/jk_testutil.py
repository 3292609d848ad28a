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


# ------------------------------------------------------------------------------------------
# Guarded device buffers: the stand-in for a memory checker.  Every buffer sits between two
# 256-byte canaries and starts out poisoned (0xFF bytes: NaN as a float, -1 as an int), so a
# write outside an output shows up as a broken canary and a read of something the library never
# wrote shows up as NaN / -1 in the results.
# ------------------------------------------------------------------------------------------
class Guard:
    PAD = 256
    CANARY = 0xA5
    POISON = 0xFF

    def __init__(self):
        self.regions = []

    def alloc(self, shape, dtype: torch.dtype) -> torch.Tensor:
        shape = tuple(int(s) for s in shape)
        n = int(np.prod(shape, dtype=np.int64)) * torch.empty((), dtype=dtype).element_size()
        body = (n + 255) // 256 * 256
        raw = torch.full((self.PAD + body + self.PAD,), self.CANARY, dtype=torch.uint8, device="cuda")
        raw[self.PAD:self.PAD + n] = self.POISON
        self.regions.append((raw, n))
        return raw[self.PAD:self.PAD + n].view(dtype).view(shape)

    def like(self, t: torch.Tensor, keep: bool = False) -> torch.Tensor:
        g = self.alloc(t.shape, t.dtype)
        if keep:
            g.copy_(t)
        return g

    def check(self):
        torch.cuda.synchronize()
        for i, (raw, n) in enumerate(self.regions):
            assert bool((raw[:self.PAD] == self.CANARY).all()), f"write before buffer {i}"
            assert bool((raw[self.PAD + n:] == self.CANARY).all()), f"write past buffer {i}"


def guarded_context(w, **kw):
    """A context whose workspace is poisoned and fenced by canaries.  Returns (ctx, check)."""
    from paper_2502_06282_b200 import binding as jk
    ctx = jk.Context.for_workload(w, allocate=False, **kw)
    n = ctx.workspace_bytes
    pad = 512
    raw = torch.full((pad + n + pad + 256,), Guard.CANARY, dtype=torch.uint8, device="cuda")
    first = (raw.data_ptr() + pad + 255) // 256 * 256 - raw.data_ptr()
    raw[first:first + n] = Guard.POISON           # poison first: jk_set_workspace then clears
    torch.cuda.synchronize()                      # the part that has to start at zero
    off = ctx.set_workspace(raw, pad)
    assert off == first

    def check():
        torch.cuda.synchronize()
        assert bool((raw[:off] == Guard.CANARY).all()), "write before the workspace"
        assert bool((raw[off + n:] == Guard.CANARY).all()), "write past the workspace"

    return ctx, check


def guarded_step_buffers(ctx, w, guard: Guard, bufs=None):
    """StepBuffers whose every tensor is a guarded, poisoned allocation."""
    from paper_2502_06282_b200 import binding as jk
    if bufs is None:
        bufs = jk.StepBuffers(ctx, w)
    for k in bufs.pool:
        bufs.pool[k] = guard.like(bufs.pool[k])
    bufs.pool_struct = ctx.pool_struct(bufs.pool)
    for name in ("probs", "expert", "gate", "feat", "frontier"):
        setattr(bufs, name, [guard.like(t) for t in getattr(bufs, name)])
    if bufs.lse_all is not None:
        bufs.lse_all = guard.like(bufs.lse_all)
        bufs.lse = bufs.lse_views()
    else:
        bufs.lse = [guard.like(t) for t in bufs.lse]
    bufs.parent_score = [guard.like(bufs.parent_score[0], keep=True)] + [
        guard.like(t) for t in bufs.parent_score[1:]]
    bufs.parent_gidx = [guard.like(bufs.parent_gidx[0], keep=True)] + [
        guard.like(t) for t in bufs.parent_gidx[1:]]
    if bufs.logits is not None:
        bufs.logits = guard.like(bufs.logits)
    bufs.tree = {k: guard.like(v) for k, v in bufs.tree.items()}
    for name in ("anc", "n_acc", "acc_idx", "acc_tok", "bonus"):
        setattr(bufs, name, guard.like(getattr(bufs, name)))
    return bufs
