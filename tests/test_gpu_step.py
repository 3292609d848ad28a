"""One whole draft-and-verify step through the C interface, as the benchmark chains it:
D x jk_draft_expand -> jk_tree_finalize -> L x jk_tree_verify_attn -> jk_accept_and_compact in
sampling mode on the library's OWN draft logits and slot numbers.

Every stage is replayed through the CPU oracle (staged replay): floating stages are compared
with the oracle's independent result by tolerance; every discrete decision is re-derived by the
oracle from the GPU's floating inputs to that decision and compared exactly.  All device buffers
are poisoned and fenced by canaries.
"""
import math

import numpy as np
import pytest
import torch

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import binding as jk
from paper_2502_06282_b200 import synth
from tests.jk_testutil import (TOL, Guard, dev, guarded_context, guarded_step_buffers, host,
                               rel_err, weights_to_device)
from tests.test_gpu_accept import _near_tie
from tests.test_gpu_expand import _check_layers, _check_tree

pytestmark = pytest.mark.gpu


def _run_step(w, mode, rows=None, heads=None, alpha=0.8):
    """rows: {layer: [(b, f), ...]} to recompute on the CPU (None = every row, small shapes
    only); heads: q heads whose attention output the oracle recomputes (None = all)."""
    tol = TOL[w.dtype]
    B, M, L, K = w.batch, w.tree_size, w.n_layers, w.top_k
    wts_np = synth.draft_weights(w)
    us_np = [synth.layer_hidden(w, l, F) for l, F in enumerate(w.frontier_sizes)]
    ctx, check_ws = guarded_context(w)
    guard = Guard()
    bufs = guarded_step_buffers(ctx, w, guard)
    wts = weights_to_device(wts_np, w.dtype)
    root = torch.full((B,), 5, dtype=torch.int32, device="cuda")
    # ---- draft
    jk.run_draft(ctx, bufs, wts, [dev(u, w.dtype) for u in us_np], root)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    if rows is None:
        pool = _check_layers(w, wts_np, us_np, bufs)
    else:
        pool = {k: host(v) for k, v in bufs.pool.items()}
        head64 = wts_np["lm_head"].astype(np.float64)
        slot_base = 0
        for l, F in enumerate(w.frontier_sizes):
            for b, f in rows.get(l, []):
                u = us_np[l][b, f].astype(np.float64)
                x = orc.rmsnorm(u, wts_np["norm_weight"], 1e-5)
                probs_o = orc.router_scores(x, wts_np["router"])
                ids, _ = orc.topk_gate(host(bufs.probs[l])[b, f], K)
                assert host(bufs.expert[l])[b, f].tolist() == ids.tolist()
                _, br, ff = orc.moe_features(u, x, ids, probs_o[ids], wts_np)
                assert rel_err(host(bufs.feat[l])[b, f], ff) <= tol
                assert rel_err(host(bufs.logits[b, slot_base + f]), br @ head64.T) <= tol
            slot_base += F
    _check_tree(w, pool, bufs, 5)
    tree_np = {k: host(v) for k, v in bufs.tree.items()}
    # ---- verify: L target layers, each on its own cache, with the tree the library built
    scale = 1.0 / math.sqrt(w.head_dim)
    caches, kds, vds = [], [], []
    kv_len_np = None
    G = w.n_q_heads // w.n_kv_heads
    for l in range(L):
        q, k, v, kv_len_np = synth.attn_inputs(w, l, ragged=True)
        caches.append((k, v))
        qd, kd, vd = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
        kds.append(kd)
        vds.append(vd)
        out = guard.like(qd)
        ctx.tree_verify_attn(B, M, qd, kd, vd, dev(kv_len_np), bufs.tree["parent"], scale, out)
        torch.cuda.synchronize()
        got = host(out)
        for h in (range(w.n_q_heads) if heads is None else heads):
            kh = h // G
            ref = orc.tree_verify_attn(q[:, :, h:h + 1], k[:, kh:kh + 1], v[:, kh:kh + 1],
                                       kv_len_np, tree_np["parent"], scale)
            assert rel_err(got[:, :, h:h + 1], ref) <= tol, (l, h)
    assert ctx.read_status() == 0
    # ---- accept on the library's own draft logits, slots and tree
    tl_np = synth.target_logits(w, tree_np["tok"], tree_np["parent"], alpha)
    ua_np, ub_np = synth.uniforms(w)
    kp = torch.tensor([t.data_ptr() for t in kds], dtype=torch.int64, device="cuda")
    vp = torch.tensor([t.data_ptr() for t in vds], dtype=torch.int64, device="cuda")
    kvl = guard.like(dev(kv_len_np), keep=True)
    ctx.accept_and_compact(B, M, mode, 1.0 if mode else 0.0, dev(tl_np), bufs.tree,
                           bufs.logits if mode else None, w.n_slots,
                           dev(ua_np) if mode else None, dev(ub_np) if mode else None, L, kp, vp,
                           kds[0].stride(0), kds[0].stride(1), kds[0].shape[2], kvl, bufs.n_acc,
                           bufs.acc_idx, bufs.acc_tok, bufs.bonus)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    guard.check()
    check_ws()
    dl_np = host(bufs.logits)
    n_acc, acc_idx, bonus = host(bufs.n_acc), host(bufs.acc_idx), host(bufs.bonus)
    paths, ties = [], 0
    for b in range(B):
        got_path = acc_idx[b, :n_acc[b]].tolist()
        if mode == 0:
            path, toks, bo = orc.accept_greedy(tl_np[b], tree_np["tok"][b], tree_np["parent"][b])
            assert got_path == path and bonus[b] == bo
        else:
            trace = []
            path, toks, bo = orc.accept_sampling(
                tl_np[b], tree_np["tok"][b], tree_np["parent"][b], tree_np["depth"][b],
                tree_np["branch"][b], tree_np["qslot"][b], dl_np[b], ua_np[b], ub_np[b], 1.0,
                trace=trace)
            if got_path != path or bonus[b] != bo:
                # fp32 on the GPU, fp64 here: only a decision within rounding of its threshold
                # may differ
                assert _near_tie(trace, ua_np[b]), (b, got_path, path, bonus[b], bo)
                ties += 1
        paths.append(got_path)
        assert host(bufs.acc_tok)[b, :len(got_path)].tolist() == tree_np["tok"][b][got_path].tolist()
        assert np.all(acc_idx[b, len(got_path):] == -1)
        assert host(kvl)[b] == kv_len_np[b] + 1 + len(got_path)
    assert ties <= 1
    for l, (k, v) in enumerate(caches):
        for b in range(B):
            assert np.array_equal(host(kds[l])[b], orc.compact_kv(k[b], int(kv_len_np[b]), paths[b]))
            assert np.array_equal(host(vds[l])[b], orc.compact_kv(v[b], int(kv_len_np[b]), paths[b]))
    return paths


@pytest.mark.parametrize("name,batch", [("tiny", 1), ("tiny_bf16", 1), ("tiny_bf16", 3)])
@pytest.mark.parametrize("mode", [0, 1])
def test_step_tiny_every_stage_replayed(name, batch, mode):
    w = synth.scaled(synth.WORKLOADS[name], batch=batch)
    _run_step(w, mode)


def test_step_llama2_7b_shape_sampling():
    """The benchmarked chain at the LLaMA2-7B shape with three target layers: all six draft
    layers, the tree the library builds, attention on it, and sampling acceptance on the
    library's own 51 x 2 draft-logit rows; one recomputed row per draft layer and three q heads
    per attention layer."""
    w = synth.scaled(synth.WORKLOADS["llama2_7b"], n_layers=3)
    rows = {0: [(0, 0)], 1: [(0, 6)], 2: [(0, 1)], 3: [(0, 9)], 4: [(0, 4)], 5: [(0, 0)]}
    _run_step(w, 1, rows=rows, heads=(0, 11, 31))
