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


def _run(w, parent_np, ragged=False, layer=0, kernel=0):
    q, k, v, kv_len = synth.attn_inputs(w, layer, ragged)
    ctx = jk.Context.for_workload(w)
    assert ctx.tensor_path_active == (w.dtype == "bf16")
    ctx.set_attn_kernel(kernel)
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


@pytest.mark.parametrize("kind", ["chain", "star", "binary", "random"])
@pytest.mark.parametrize("kernel", [1, 2, 3])
def test_attn_tiny_every_tensor_core_kernel(kind, kernel):
    w = synth.WORKLOADS["tiny_bf16"]
    got, ref = _run(w, _trees(w, kind), kernel=kernel)
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
    (8192, 128, 8, 2, 128, 2),    # the longest prefix and largest tree of the sweep: 65 key tiles
    (4096, 64, 8, 8, 64, 8),      # batch 8, ragged lengths, head size 64
    (512, 60, 32, 8, 64, 4),      # 7680 output rows, head size 64: the persistent kernel's merge
                                  # takes two rows per warp
    (200, 57, 45, 45, 128, 3),    # 7695 rows (odd: the last warp of that merge has one live row)
])
def test_attn_shapes(dtype, P, M, Hq, Hkv, d, B):
    w = synth.scaled(synth.WORKLOADS["tiny"], name="attn", dtype=dtype, prefix=P, tree_size=M,
                     n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, batch=B, depth=6,
                     seed=900 + P + M)
    # bf16: every tensor-core kernel (1 = CTA per key slice, 2 = persistent, 3 = cluster-merged);
    # f32: CUDA cores
    for kernel in ((1, 2, 3) if dtype == "bf16" else (0,)):
        got, ref = _run(w, _trees(w, "random"), ragged=True, kernel=kernel)
        assert rel_err(got, ref) <= TOL[dtype], kernel


@pytest.mark.parametrize("name,heads,ragged", [
    ("llama2_7b", (0, 13, 31), False),          # benchmark shape: MHA 32 x 128, P = 1024
    ("llama2_13b_b4", (5, 39), True),           # batch 4 with ragged prefix lengths, P <= 2048
    ("llama3_8b", (0, 17), False),              # GQA 32/8, P = 4096: two query blocks per kv head
    ("llama2_70b_layer", (9, 63), False),       # GQA 64/8, P = 4096: four query blocks per kv head
])
@pytest.mark.parametrize("kernel", [0, 1, 2, 3])
def test_attn_full_shapes_sampled_heads(name, heads, ragged, kernel):
    """Full-size shapes (0 = the kernel the library picks, as benchmarked; 1, 2, 3 = each kernel
    forced); the oracle checks a few q heads."""
    w = synth.WORKLOADS[name]
    par = _trees(w, "random")
    q, k, v, kv_len = synth.attn_inputs(w, 0, ragged)
    ctx = jk.Context.for_workload(w)
    assert ctx.tensor_path_active
    ctx.set_attn_kernel(kernel)
    qd, kd, vd = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
    out = torch.empty_like(qd)
    ctx.tree_verify_attn(w.batch, w.tree_size, qd, kd, vd, dev(kv_len), dev(par),
                         1.0 / math.sqrt(w.head_dim), out)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    got = host(out)
    G = w.n_q_heads // w.n_kv_heads
    for h in heads:
        kh = h // G
        ref = orc.tree_verify_attn(q[:, :, h:h + 1], k[:, kh:kh + 1], v[:, kh:kh + 1], kv_len,
                                   par, 1.0 / math.sqrt(w.head_dim))
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


@pytest.mark.parametrize("kernel", [2, 3])
def test_attn_tensor_core_kernels_report_a_cache_that_is_too_short(kernel):
    w = synth.WORKLOADS["tiny_bf16"]
    q, k, v, kv_len = synth.attn_inputs(w)
    ctx = jk.Context.for_workload(w)
    ctx.set_attn_kernel(kernel)
    qd, kd, vd = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
    out = torch.zeros_like(qd)
    bad_len = dev(np.array([k.shape[2] - w.tree_size + 1] * w.batch, dtype=np.int32))
    ctx.tree_verify_attn(w.batch, w.tree_size, qd, kd, vd, bad_len, dev(_trees(w, "chain")),
                         0.125, out)
    assert ctx.read_status() == jk.ERR["BOUNDS"]
    assert ctx.read_status() == 0


@pytest.mark.parametrize("kernel", [1, 2, 3])
def test_attn_is_bitwise_reproducible(kernel):
    """Slices are merged in a fixed order: two calls on the same inputs give the same bits."""
    w = synth.scaled(synth.WORKLOADS["tiny"], name="attn", dtype="bf16", prefix=1500, tree_size=60,
                     n_q_heads=32, n_kv_heads=8, head_dim=128, batch=2, depth=6, seed=77)
    q, k, v, kv_len = synth.attn_inputs(w, 0, True)
    ctx = jk.Context.for_workload(w)
    ctx.set_attn_kernel(kernel)
    qd, kd, vd = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
    par, kvd = dev(_trees(w, "random")), dev(kv_len)
    outs = []
    for _ in range(2):
        out = torch.empty_like(qd)
        ctx.tree_verify_attn(w.batch, w.tree_size, qd, kd, vd, kvd, par, 1.0 / math.sqrt(w.head_dim), out)
        torch.cuda.synchronize()
        outs.append(out.view(torch.int16).cpu())
    assert ctx.read_status() == 0
    assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("dtype,kernel", [("f32", 0), ("bf16", 0), ("bf16", 1), ("bf16", 2),
                                          ("bf16", 3)])
def test_attn_ignores_cache_rows_past_the_tree(dtype, kernel):
    """The operation is defined over cache rows c < kv_len + M only (Sec. 2.1 step 2).  Rows
    between kv_len + M and the cache capacity belong to nobody: here they hold NaN (as a pool
    that was never cleared may), in K and in V, and must leave no trace in the output.  Ragged
    lengths put the dead rows in the middle of a key tile for some sequences and make a whole
    tile dead for others."""
    w = synth.scaled(synth.WORKLOADS["tiny"], name="attn_nan", dtype=dtype, prefix=300,
                     tree_size=37, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=3, depth=6,
                     seed=4711)
    par = _trees(w, "random")
    q, k, v, kv_len = synth.attn_inputs(w, 0, ragged=True)
    kv_len[1] = 90                                     # one sequence leaves two whole tiles dead
    k, v = k.copy(), v.copy()
    for b in range(w.batch):
        k[b, :, int(kv_len[b]) + w.tree_size:] = np.nan
        v[b, :, int(kv_len[b]) + w.tree_size:] = np.nan
    assert np.isnan(k).any()
    ctx = jk.Context.for_workload(w)
    ctx.set_attn_kernel(kernel)
    kd = torch.from_numpy(k).cuda()
    vd = torch.from_numpy(v).cuda()
    if dtype == "bf16":
        kd, vd = kd.to(torch.bfloat16), vd.to(torch.bfloat16)
    qd = dev(q, w.dtype)
    out = torch.empty_like(qd)
    scale = 1.0 / math.sqrt(w.head_dim)
    ctx.tree_verify_attn(w.batch, w.tree_size, qd, kd, vd, dev(kv_len), dev(par), scale, out)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    got = host(out)
    assert not np.isnan(got).any()
    ref = orc.tree_verify_attn(q, np.nan_to_num(k), np.nan_to_num(v), kv_len, par, scale)
    assert rel_err(got, ref) <= TOL[dtype]
