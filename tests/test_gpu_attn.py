"""GPU parity of jk_tree_verify_attn against the oracle's plain masked attention."""
import math

import numpy as np
import pytest
import torch

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import binding as jk
from paper_2502_06282_b200 import synth
from tests.jk_testutil import TOL, dev, host, rel_err

pytestmark = pytest.mark.gpu


def _run(w, parent_np, ragged=False, layer=0):
    q, k, v, kv_len = synth.attn_inputs(w, layer, ragged)
    ctx = jk.Context.for_workload(w)
    assert ctx.tensor_path_active == (w.dtype == "bf16")
    qd, kd, vd = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
    out = torch.empty_like(qd)
    ctx.tree_verify_attn(w.batch, w.tree_size, qd, kd, vd, dev(kv_len), dev(parent_np),
                         1.0 / math.sqrt(w.head_dim), out)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    ref = orc.tree_verify_attn(q, k, v, kv_len, parent_np, 1.0 / math.sqrt(w.head_dim))
    return host(out), ref


def _trees(w, kind):
    M, B = w.tree_size, w.batch
    if kind == "chain":
        p = synth.chain_tree(M)
    elif kind == "star":
        p = synth.star_tree(M)
    elif kind == "binary":
        p = synth.binary_tree(M)
    else:
        return np.stack([synth.random_tree(M, w.depth, w.seed + b) for b in range(B)])
    return np.stack([p] * B)


@pytest.mark.parametrize("name", ["tiny", "tiny_bf16"])
@pytest.mark.parametrize("kind", ["chain", "star", "binary", "random"])
def test_attn_tiny(name, kind):
    w = synth.WORKLOADS[name]
    got, ref = _run(w, _trees(w, kind))
    assert rel_err(got, ref) <= TOL[w.dtype]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("P,M,Hq,Hkv,d,B", [
    (0, 1, 2, 2, 64, 1),          # empty prefix, single node
    (1, 5, 4, 1, 128, 2),         # one prefix token, all q heads on one kv head
    (37, 13, 8, 2, 128, 3),       # ragged tiles, GQA 4
    (300, 128, 4, 4, 64, 1),      # the largest tree
    (777, 60, 16, 2, 128, 2),     # GQA 8: several query blocks per kv head
    (1500, 60, 32, 32, 128, 2),   # many heads: each CTA walks several key tiles (running max)
    (900, 33, 16, 16, 64, 3),     # the same with head size 64
])
def test_attn_shapes(dtype, P, M, Hq, Hkv, d, B):
    w = synth.scaled(synth.WORKLOADS["tiny"], name="attn", dtype=dtype, prefix=P, tree_size=M,
                     n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, batch=B, depth=6,
                     seed=900 + P + M)
    got, ref = _run(w, _trees(w, "random"), ragged=True)
    assert rel_err(got, ref) <= TOL[dtype]


def test_attn_llama2_7b_shape_sampled_heads():
    """Benchmark shape (32 heads x 128, P = 1024, M = 60); the oracle checks three heads."""
    w = synth.WORKLOADS["llama2_7b"]
    par = _trees(w, "random")
    q, k, v, kv_len = synth.attn_inputs(w, 0)
    ctx = jk.Context.for_workload(w)
    qd, kd, vd = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
    out = torch.empty_like(qd)
    ctx.tree_verify_attn(1, w.tree_size, qd, kd, vd, dev(kv_len), dev(par),
                         1.0 / math.sqrt(w.head_dim), out)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    got = host(out)
    for h in (0, 13, 31):
        ref = orc.tree_verify_attn(q[:, :, h:h + 1], k[:, h:h + 1], v[:, h:h + 1], kv_len, par,
                                   1.0 / math.sqrt(w.head_dim))
        assert rel_err(got[:, :, h:h + 1], ref) <= TOL[w.dtype]


def test_attn_reports_a_cache_that_is_too_short():
    w = synth.WORKLOADS["tiny"]
    q, k, v, kv_len = synth.attn_inputs(w)
    ctx = jk.Context.for_workload(w)
    qd, kd, vd = dev(q), dev(k), dev(v)
    out = torch.zeros_like(qd)
    bad_len = dev(np.array([k.shape[2] - w.tree_size + 1], dtype=np.int32))
    ctx.tree_verify_attn(1, w.tree_size, qd, kd, vd, bad_len, dev(_trees(w, "chain")), 0.125, out)
    assert ctx.read_status() == jk.ERR["BOUNDS"]
    assert ctx.read_status() == 0          # reading clears it
