"""jk_tree_verify_attn_static: tree attention for callers that cannot allocate.

Some users of this library reserve all of the GPU's memory for their own pools when they start
(an inference server sizing its KV cache to whatever is free), or run a decode loop in which the
device-wide stall of cudaMalloc/cudaFree is not acceptable.  They cannot hand the library a
workspace, so this entry point keeps its split-KV partials in an 8 MiB array built into the
library.  The test calls it through the C interface without ever setting a workspace and checks
the result against jk_tree_verify_attn, twice in a row with different inputs, because the array
is shared by all calls and still holds the previous call's partials on the second one.

Collected last on purpose (file name): a failure here must not hide other tests' results.
"""
import math

import numpy as np
import pytest
import torch

from paper_2502_06282_b200 import binding as jk
from paper_2502_06282_b200 import synth
from tests.jk_testutil import TOL, dev, host, rel_err

pytestmark = pytest.mark.gpu


def _inputs(w, layer, tree_seed):
    q, k, v, kv_len = synth.attn_inputs(w, layer, ragged=True)
    parent = np.stack([synth.random_tree(w.tree_size, w.depth, tree_seed + b)
                       for b in range(w.batch)])
    return (dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype), dev(kv_len), dev(parent))


@pytest.mark.parametrize("name,batch", [("tiny", 2), ("tiny_bf16", 1)])
def test_static_scratch_attention_matches_the_workspace_version(name, batch):
    w = synth.scaled(synth.WORKLOADS[name], batch=batch, prefix=333)
    scale = 1.0 / math.sqrt(w.head_dim)
    ref_ctx = jk.Context.for_workload(w)                       # ordinary path, with workspace
    bare_ctx = jk.Context.for_workload(w, allocate=False)      # never gets a workspace
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for call, (layer, tree_seed) in enumerate([(0, 40), (1, 50)]):
        q, k, v, kv_len, parent = _inputs(w, layer, tree_seed)
        want = torch.empty_like(q)
        ref_ctx.tree_verify_attn(w.batch, w.tree_size, q, k, v, kv_len, parent, scale, want)
        got = torch.full_like(q, float("nan"))
        bare_ctx.tree_verify_attn_static(w.batch, w.tree_size, q, k, v, kv_len, parent, scale,
                                         got, status if call == 0 else None)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        assert rel_err(host(got), host(want)) <= TOL[w.dtype], f"call {call}"


def test_static_scratch_rejects_sizes_beyond_its_array():
    # 8 sequences x 128 nodes x 64 heads x (128 + 2) floats = 34 MB of partials per key slice
    w = synth.scaled(synth.WORKLOADS["tiny_bf16"], batch=8, tree_size=128, n_q_heads=64,
                     n_kv_heads=8, head_dim=128)
    ctx = jk.Context.for_workload(w, allocate=False)
    q = torch.zeros(8, 128, 64, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(8, 8, 256, 128, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(8, 128, dtype=torch.int32, device="cuda")
    with pytest.raises(jk.JakiroError) as e:
        ctx.tree_verify_attn_static(8, 128, q, kv, kv, idx, idx, 1.0, torch.empty_like(q))
    assert e.value.code == jk.ERR["CAPACITY"] and "built-in scratch" in str(e.value)
