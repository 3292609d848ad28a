"""jk_tree_verify_attn_static: tree attention for callers that cannot allocate.

Some users of this library reserve all of the GPU's memory for their own pools when they start
(an inference server sizing its KV cache to whatever is free), or run a decode loop in which the
device-wide stall of cudaMalloc/cudaFree is not acceptable.  They cannot hand the library a
workspace, so this entry point keeps its split-KV partials in an 8 MiB array built into the
library.  The tests call it through the C interface without ever setting a workspace and check
the result against jk_tree_verify_attn and against the CPU oracle, twice in a row: the array is
shared by all calls and on the second call still holds the first call's partials, and the second
call is the smaller one (fewer key slices), so a stale partial that was read would show.

Collected last on purpose (file name): a failure here must not hide other tests' results.
"""
import math

import numpy as np
import pytest
import torch

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import binding as jk
from paper_2502_06282_b200 import synth
from tests.jk_testutil import TOL, dev, host, rel_err

pytestmark = pytest.mark.gpu


def _inputs(w, layer, tree_seed):
    q, k, v, kv_len = synth.attn_inputs(w, layer, ragged=True)
    parent = np.stack([synth.random_tree(w.tree_size, w.depth, tree_seed + b)
                       for b in range(w.batch)])
    return q, k, v, kv_len, parent


@pytest.mark.parametrize("name,batch", [("tiny", 2), ("tiny_bf16", 1)])
def test_static_scratch_attention_matches_the_workspace_version_and_the_oracle(name, batch):
    base = synth.scaled(synth.WORKLOADS[name], batch=batch, prefix=333)
    scale = 1.0 / math.sqrt(base.head_dim)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # second call: shorter prefix and a smaller tree, so fewer and smaller partials
    for call, w in enumerate([base, synth.scaled(base, prefix=40, tree_size=9, seed=base.seed + 1)]):
        ref_ctx = jk.Context.for_workload(w)                       # ordinary path, with workspace
        bare_ctx = jk.Context.for_workload(w, allocate=False)      # never gets a workspace
        q, k, v, kv_len, parent = _inputs(w, call, 40 + 10 * call)
        qd, kd, vd = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
        kvd, pd = dev(kv_len), dev(parent)
        want = torch.empty_like(qd)
        ref_ctx.tree_verify_attn(w.batch, w.tree_size, qd, kd, vd, kvd, pd, scale, want)
        got = torch.full_like(qd, float("nan"))
        bare_ctx.tree_verify_attn_static(w.batch, w.tree_size, qd, kd, vd, kvd, pd, scale, got,
                                         status)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        assert rel_err(host(got), host(want)) <= TOL[w.dtype], f"call {call}"
        ref = orc.tree_verify_attn(q, k, v, kv_len, parent, scale)
        assert rel_err(host(got), ref) <= TOL[w.dtype], f"call {call} against the oracle"


def test_static_scratch_reports_a_cache_that_is_too_short():
    w = synth.WORKLOADS["tiny"]
    q, k, v, kv_len, parent = _inputs(w, 0, 60)
    ctx = jk.Context.for_workload(w, allocate=False)
    qd, kd, vd = dev(q), dev(k), dev(v)
    out = torch.zeros_like(qd)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bad_len = dev(np.array([k.shape[2] - w.tree_size + 1], dtype=np.int32))
    ctx.tree_verify_attn_static(1, w.tree_size, qd, kd, vd, bad_len, dev(parent), 0.125, out,
                                status)
    torch.cuda.synchronize()
    assert int(status[0]) == jk.ERR["BOUNDS"]
    # and a missing status word is an argument error, before anything is launched
    with pytest.raises(jk.JakiroError) as e:
        ctx.tree_verify_attn_static(1, w.tree_size, qd, kd, vd, dev(kv_len), dev(parent), 0.125,
                                    out, None)
    assert e.value.code == jk.ERR["NULL"]


def test_static_scratch_rejects_sizes_beyond_its_array():
    # 8 sequences x 128 nodes x 64 heads x (128 + 2) floats = 34 MB of partials per key slice
    w = synth.scaled(synth.WORKLOADS["tiny_bf16"], batch=8, tree_size=128, n_q_heads=64,
                     n_kv_heads=8, head_dim=128)
    ctx = jk.Context.for_workload(w, allocate=False)
    q = torch.zeros(8, 128, 64, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(8, 8, 256, 128, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(8, 128, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(jk.JakiroError) as e:
        ctx.tree_verify_attn_static(8, 128, q, kv, kv, idx, idx, 1.0, torch.empty_like(q), status)
    assert e.value.code == jk.ERR["CAPACITY"] and "built-in scratch" in str(e.value)
