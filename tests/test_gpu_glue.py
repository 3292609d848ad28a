"""GPU parity of the verification-side glue (Sec. 2.1 step 2-3): jk_verify_qkv (QKV projection of
the tree tokens, rotary positions by depth, K/V written at the tree slots), the attention it
feeds, and jk_gather_accepted (the accepted path's hidden states for the next draft round)."""
import math

import numpy as np
import pytest
import torch

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import binding as jk
from paper_2502_06282_b200 import synth
from tests.jk_testutil import TOL, Guard, dev, guarded_context, host, rel_err

pytestmark = pytest.mark.gpu
THETA = 10000.0


def _case(w, tensor_path=None):
    ctx, check_ws = guarded_context(w)
    if tensor_path is not None:
        ctx.set_tensor_path(tensor_path)
    guard = Guard()
    B, M, H = w.batch, w.tree_size, w.hidden
    qd, kvd = w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim
    w_qkv = synth.pre_weights(w)["w_qkv"]
    rng = np.random.default_rng(w.seed)
    x = synth.store_round(rng.standard_normal((B, M, H)).astype(np.float32), w.dtype)
    parent = np.stack([synth.random_tree(M, w.depth, w.seed + b) for b in range(B)])
    depth = np.stack([synth.tree_depths(p) for p in parent])
    _, k0, v0, kv_len = synth.attn_inputs(w, 0, ragged=True)
    kd, vd = dev(k0, w.dtype), dev(v0, w.dtype)
    q_out = guard.alloc((B, M, w.n_q_heads, w.head_dim), ctx.tdtype)
    ctx.verify_qkv(dev(w_qkv, w.dtype), B, M, dev(x, w.dtype), dev(depth), q_out, kd, vd,
                   dev(kv_len), THETA)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    guard.check()
    check_ws()
    tol = TOL[w.dtype]
    for b in range(B):
        P = int(kv_len[b])
        q_o, kc, vc = orc.verify_qkv_append(x[b], w_qkv[:qd], w_qkv[qd:qd + kvd], w_qkv[qd + kvd:],
                                            depth[b], k0[b], v0[b], P, w.n_q_heads, w.n_kv_heads, THETA)
        assert rel_err(host(q_out)[b], q_o) <= tol
        assert rel_err(host(kd)[b][:, P:P + M], kc[:, P:P + M]) <= tol
        assert rel_err(host(vd)[b][:, P:P + M], vc[:, P:P + M]) <= tol
        keep = np.ones(k0.shape[2], dtype=bool)
        keep[P:P + M] = False
        assert np.array_equal(host(kd)[b][:, keep], k0[b][:, keep])
    # and the attention on what the call wrote (staged: the oracle attends over the GPU's q, K, V)
    out = torch.empty_like(q_out)
    scale = 1.0 / math.sqrt(w.head_dim)
    ctx.tree_verify_attn(B, M, q_out, kd, vd, dev(kv_len), dev(parent), scale, out)
    torch.cuda.synchronize()
    ref = orc.tree_verify_attn(host(q_out), host(kd), host(vd), kv_len, parent, scale)
    assert rel_err(host(out), ref) <= tol
    return ctx


@pytest.mark.parametrize("name,tensor_path", [("tiny", None), ("tiny_bf16", False),
                                              ("tiny_bf16", True)])
def test_verify_qkv_and_attention(name, tensor_path):
    w = synth.scaled(synth.WORKLOADS[name], batch=2, n_q_heads=8, n_kv_heads=2, prefix=150, seed=7070)
    _case(w, tensor_path)


def test_verify_qkv_more_than_256_tree_tokens():
    # 3 sequences x 100 nodes = 300 rows: two passes of the projection GEMM
    w = synth.scaled(synth.WORKLOADS["tiny_bf16"], batch=3, tree_size=100, depth=8, prefix=64,
                     seed=7171)
    ctx = _case(w)
    assert ctx.tensor_path_active


def test_verify_qkv_llama2_7b_shape():
    w = synth.scaled(synth.WORKLOADS["llama2_7b"], seed=7272)
    _case(w)


def test_gather_accepted():
    w = synth.scaled(synth.WORKLOADS["tiny_bf16"], batch=3)
    ctx = jk.Context.for_workload(w)
    B, M, H, D = w.batch, w.tree_size, w.hidden, w.depth
    rng = np.random.default_rng(5)
    hidden = synth.store_round(rng.standard_normal((B, M, H)).astype(np.float32), w.dtype)
    n_acc = np.array([0, 2, D], dtype=np.int32)
    acc_idx = np.full((B, D), -1, dtype=np.int32)
    acc_idx[1, :2] = [3, 9]
    acc_idx[2] = [1, 4, 7, 15]
    guard = Guard()
    out = guard.alloc((B, D + 1, H), ctx.tdtype)
    ctx.gather_accepted(B, M, dev(hidden, w.dtype), dev(n_acc), dev(acc_idx), D + 1, out)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    guard.check()
    for b in range(B):
        want = orc.gather_accepted(hidden[b], acc_idx[b, :n_acc[b]], D + 1)
        assert np.array_equal(host(out)[b], want)
