"""GPU parity of jk_draft_pre (the draft layer in front of the MoE: Sec. 3.1.2, Eq. 1) and of the
chained draft jk_draft_pre -> jk_draft_expand -> ... against the CPU oracle.  Staged replay: the
oracle recomputes every pass from the GPU's own inputs to that pass (tokens from the pool, parent
features from the previous jk_draft_expand) and keeps its own fp64 copy of the draft layer's KV
cache from pass to pass."""
import math

import numpy as np
import pytest
import torch

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import binding as jk
from paper_2502_06282_b200 import synth
from tests.jk_testutil import (TOL, Guard, dev, guarded_context, guarded_step_buffers, host,
                               rel_err, weights_to_device)
from tests.test_gpu_expand import _check_layers, _check_tree

pytestmark = pytest.mark.gpu
THETA = 10000.0


def _split_pre(pw, w):
    qd, kvd = w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim
    out = {"emb": pw["emb"], "w_fc": pw["w_fc"], "b_fc": pw.get("b_fc"), "w_o": pw["w_o"],
           "w_q": pw["w_qkv"][:qd], "w_k": pw["w_qkv"][qd:qd + kvd], "w_v": pw["w_qkv"][qd + kvd:]}
    return out


def _ancestors(slot_parent, s):
    while s >= 0:
        yield s
        s = int(slot_parent[s])


def _run_chained(w, tensor_path=None, bias=True, layer_id=90):
    ctx, check_ws = guarded_context(w)
    if tensor_path is not None:
        ctx.set_tensor_path(tensor_path)
        assert ctx.tensor_path_active == bool(tensor_path)
    guard = Guard()
    bufs = guarded_step_buffers(ctx, w, guard)
    pre = jk.PreBuffers(ctx, bufs)
    wts_np = synth.draft_weights(w)
    pw_np = synth.pre_weights(w, bias)
    root_feat = synth.root_feature(w)
    _, k0, v0, kv_len = synth.attn_inputs(w, layer_id, ragged=True)
    kd, vd = dev(k0, w.dtype), dev(v0, w.dtype)
    root = torch.full((w.batch,), 5, dtype=torch.int32, device="cuda")
    scale = 1.0 / math.sqrt(w.head_dim)
    jk.run_draft_chained(ctx, bufs, pre, weights_to_device(wts_np, w.dtype),
                         weights_to_device(pw_np, w.dtype), root, dev(root_feat, w.dtype), kd, vd,
                         dev(kv_len), THETA, scale)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    guard.check()
    check_ws()
    return ctx, bufs, pre, wts_np, pw_np, root_feat, (k0, v0, kv_len, kd, vd), scale


def _check_pre(w, bufs, pre, pw_np, root_feat, caches, scale):
    tol = TOL[w.dtype]
    k0, v0, kv_len, kd, vd = caches
    pw = _split_pre(pw_np, w)
    fs = bufs.frontier_sizes
    K, ke = w.top_k, w.k_per_expert
    pool = {k: host(v) for k, v in bufs.pool.items()}
    sp_g, sd_g = host(pre.slot_parent), host(pre.slot_depth)
    for b in range(w.batch):
        P = int(kv_len[b])
        kc, vc = k0[b].astype(np.float64), v0[b].astype(np.float64)
        slot_parent = np.full(bufs.n_slots, -1, dtype=np.int64)
        gidx_base, slot_base = 0, 0
        prev = None
        for l, F in enumerate(fs):
            slots = list(range(slot_base, slot_base + F))
            if l == 0:
                tok = np.array([5])
                f_prev = root_feat[b][None].astype(np.float64)
            else:
                g = host(bufs.parent_gidx[l])[b]
                tok = pool["tok"][b, g]
                rows = (g - prev[0]) // (K * ke)
                f_prev = host(bufs.feat[l - 1])[b, rows].astype(np.float64)   # the GPU's own features
                slot_parent[slots] = prev[1] + rows
            u_o, h_o, kc, vc = orc.draft_pre_block(tok, f_prev, pw, kc, vc, P, slots, slot_parent,
                                                   w.n_q_heads, w.n_kv_heads, THETA, scale)
            assert sp_g[b, slots].tolist() == slot_parent[slots].tolist()
            u_g = host(pre.u[l])[b]
            if w.dtype == "f32":
                assert rel_err(u_g, u_o) <= tol, (b, l)
            else:
                # bf16 keeps h, q, k, v and the attention output in bf16 between the block's
                # stages, and a peaked softmax amplifies the rounding of q and k: the block is
                # replayed stage by stage.  Stage 1-2: the projections (q below, k and v through
                # the cache rows at the end).  Stage 3: attention and output projection
                # recomputed from the GPU's own q, k, v.
                M_l = slot_base + F
                q_g = host(pre.q)[b, :M_l].astype(np.float64)
                for i, s_ in enumerate(slots):
                    pos = P + int(np.sum([1 for _ in _ancestors(slot_parent, s_)])) - 1
                    q_o = (np.asarray(pw["w_q"], np.float64) @ h_o[i]).reshape(w.n_q_heads, -1)
                    q_o = np.stack([orc.rope(q_o[hh], pos, THETA) for hh in range(w.n_q_heads)])
                    assert rel_err(q_g[s_], q_o) <= tol, (b, l, "q")
                att = orc.tree_verify_attn(q_g[None], host(kd)[b][None], host(vd)[b][None],
                                           np.array([P]), slot_parent[None, :M_l], scale)
                u_r = att[0, slots].reshape(F, -1) @ np.asarray(pw["w_o"], np.float64).T + h_o
                assert rel_err(u_g, u_r) <= tol, (b, l, "attention + output projection")
                # End to end against the oracle's own chain: three bf16 stages through a peaked
                # softmax turn one flipped rounding of q into a visible difference of u, so this
                # is only a sanity bound; the per-stage checks above are the parity criterion.
                assert rel_err(u_g, u_o) <= 0.25, (b, l)
            prev = (gidx_base, slot_base, F)
            gidx_base += F * K * ke
            slot_base += F
        depth = np.zeros(bufs.n_slots, dtype=np.int64)
        for s in range(1, bufs.n_slots):
            depth[s] = depth[slot_parent[s]] + 1
        assert sd_g[b].tolist() == depth.tolist()
        # the draft layer's cache: this step's rows against the oracle's, every other row untouched
        S = bufs.n_slots
        assert rel_err(host(kd)[b][:, P:P + S], kc[:, P:P + S]) <= tol
        assert rel_err(host(vd)[b][:, P:P + S], vc[:, P:P + S]) <= tol
        keep = np.ones(k0.shape[2], dtype=bool)
        keep[P:P + S] = False
        assert np.array_equal(host(kd)[b][:, keep], k0[b][:, keep])
        assert np.array_equal(host(vd)[b][:, keep], v0[b][:, keep])


@pytest.mark.parametrize("name,tensor_path", [("tiny", None), ("tiny_bf16", False),
                                              ("tiny_bf16", True)])
def test_chained_draft_pre_and_expand(name, tensor_path):
    w = synth.scaled(synth.WORKLOADS[name], batch=2, n_q_heads=8, n_kv_heads=4, prefix=200, seed=6060)
    ctx, bufs, pre, wts_np, pw_np, root_feat, caches, scale = _run_chained(w, tensor_path)
    _check_pre(w, bufs, pre, pw_np, root_feat, caches, scale)
    # and the MoE passes on the hidden states the block produced
    us = [host(u) for u in pre.u]
    pool = _check_layers(w, wts_np, us, bufs)
    _check_tree(w, pool, bufs, 5)


def test_draft_pre_far_positions_and_no_bias():
    # position ~5000: the rotation angle needs more than fp32 to stay within the f32 tolerance
    w = synth.scaled(synth.WORKLOADS["tiny"], prefix=5000, depth=3, tree_size=10, seed=6161)
    ctx, bufs, pre, wts_np, pw_np, root_feat, caches, scale = _run_chained(w, bias=False)
    _check_pre(w, bufs, pre, pw_np, root_feat, caches, scale)


def test_draft_pre_llama2_7b_shape():
    """Benchmark shape (hidden 4096, 32 heads x 128, vocabulary 32000), three passes with frontier
    sizes 1, 10, 10 on the tensor-core path; every node of every pass replayed."""
    w = synth.scaled(synth.WORKLOADS["llama2_7b"], depth=3, tree_size=20)
    ctx, bufs, pre, wts_np, pw_np, root_feat, caches, scale = _run_chained(w)
    assert ctx.tensor_path_active
    _check_pre(w, bufs, pre, pw_np, root_feat, caches, scale)


def test_draft_pre_reports_a_token_outside_the_vocabulary():
    w = synth.WORKLOADS["tiny"]
    ctx = jk.Context.for_workload(w)
    bufs = jk.StepBuffers(ctx, w)
    pre = jk.PreBuffers(ctx, bufs)
    pw = weights_to_device(synth.pre_weights(w), w.dtype)
    _, k0, v0, kv_len = synth.attn_inputs(w, 90)
    bad_root = torch.full((1,), w.vocab, dtype=torch.int32, device="cuda")
    ctx.draft_pre(pw, pre.state, 1, 1, 0, None, bufs.pool_struct, 0, 0, 1,
                  dev(synth.root_feature(w)), bad_root, dev(k0), dev(v0), dev(kv_len), THETA, 0.125,
                  pre.u[0])
    assert ctx.read_status() == jk.ERR["BOUNDS"]
