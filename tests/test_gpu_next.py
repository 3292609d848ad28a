"""GPU parity of the static tree policy (Sec. 3.1.2, last paragraph) and of the contrastive heads
with the hybrid schedule (Sec. 3.2, Eq. 6-8) against the CPU oracle, through the C interface.
Staged replay as everywhere: floating stages by tolerance against the oracle's own result,
discrete decisions re-derived by the oracle from the GPU's floating inputs and compared exactly."""
import numpy as np
import pytest
import torch

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import binding as jk
from paper_2502_06282_b200 import synth
from paper_2502_06282_b200.static_tree import plan_from_paths
from tests.jk_testutil import (TOL, Guard, dev, guarded_context, guarded_step_buffers, host,
                               rel_err, weights_to_device)

pytestmark = pytest.mark.gpu

PATHS = [(0,), (1,), (3,), (0, 0), (0, 2), (3, 1), (0, 0, 3), (0, 0, 0), (3, 1, 1), (3, 1, 2)]


def _draft(w, ctx_kw, fs, static_plan=None, tensor_path=None):
    ctx, check_ws = guarded_context(w, frontier_sizes=fs, **ctx_kw)
    if tensor_path is not None:
        ctx.set_tensor_path(tensor_path)
        assert ctx.tensor_path_active == bool(tensor_path)
    guard = Guard()
    bufs = jk.StepBuffers(ctx, w, frontier_sizes=fs)
    bufs = guarded_step_buffers(ctx, w, guard, bufs)
    wts_np = synth.draft_weights(w)
    us_np = [synth.layer_hidden(w, l, F) for l, F in enumerate(fs)]
    root = torch.full((w.batch,), 5, dtype=torch.int32, device="cuda")
    jk.run_draft(ctx, bufs, weights_to_device(wts_np, w.dtype), [dev(u, w.dtype) for u in us_np],
                 root, static_plan=static_plan)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    guard.check()
    check_ws()
    return ctx, bufs, wts_np, us_np


@pytest.mark.parametrize("name,tensor_path", [("tiny", None), ("tiny_bf16", False),
                                              ("tiny_bf16", True)])
def test_static_tree_policy(name, tensor_path):
    K, ke = 2, 2
    plan = plan_from_paths(PATHS, K, ke)
    fs = plan["frontier_sizes"]
    w = synth.scaled(synth.WORKLOADS[name], batch=2, k_per_expert=ke, depth=len(fs),
                     tree_size=len(PATHS) + 1, width=max(fs), seed=321)
    dplan = {"select": [dev(np.asarray(s, np.int32)) for s in plan["select"]],
             "keep": dev(np.asarray(plan["keep"], np.int32))}
    ctx, bufs, wts_np, us_np = _draft(w, {}, fs, dplan, tensor_path)
    tol = TOL[w.dtype]
    logits = host(bufs.logits)
    # frontier order within a pass is ascending path order
    expanded = [[()]] + [[p for p in plan["order"] if len(p) == d and any(q[:-1] == p for q in PATHS)]
                         for d in range(1, len(fs))]
    slot_of, s = {}, 0
    for nodes in expanded:
        for p in nodes:
            slot_of[p] = s
            s += 1
    for b in range(w.batch):
        u_of = {p: us_np[len(p)][b, f] for nodes in expanded for f, p in enumerate(nodes)}
        t = orc.grow_static_tree(lambda p: u_of[p], wts_np, PATHS, ke, root_tok=5)
        # the shape: exactly the predefined one
        for key in ("parent", "depth", "branch"):
            assert host(bufs.tree[key])[b].tolist() == t[key].tolist(), key
        tok_g = host(bufs.tree["tok"])[b]
        assert tok_g[0] == 5
        # expanded nodes: logits against the oracle's, tokens and scores replayed from the GPU's
        score_of = {(): 0.0}
        for i, p in enumerate(t["order"]):
            if not p:
                continue
            par = p[:-1]
            lg = logits[b, slot_of[par]]
            assert rel_err(lg, t["logits"][par]) <= tol
            r, j = divmod(p[-1], ke)
            ids, sc, _ = orc.branch_topk(lg[r], ke, score_of[par])
            assert tok_g[i] == ids[j], (b, p)
            score_of[p] = float(sc[j])
            assert host(bufs.tree["qslot"])[b, i] == slot_of.get(p, -1)
        if w.dtype == "f32":
            assert tok_g.tolist() == t["tok"].tolist()        # no near-ties in this seeded case


def test_static_tree_rejects_a_bad_list():
    K, ke = 2, 2
    plan = plan_from_paths(PATHS, K, ke)
    fs = plan["frontier_sizes"]
    w = synth.scaled(synth.WORKLOADS["tiny"], k_per_expert=ke, depth=len(fs),
                     tree_size=len(PATHS) + 1, width=max(fs))
    ctx = jk.Context.for_workload(w, frontier_sizes=fs)
    bufs = jk.StepBuffers(ctx, w, frontier_sizes=fs)
    wts = weights_to_device(synth.draft_weights(w), w.dtype)
    us = [dev(synth.layer_hidden(w, l, F), w.dtype) for l, F in enumerate(fs)]
    root = torch.full((1,), 5, dtype=torch.int32, device="cuda")
    bad_sel = [dev(np.asarray([0, 99], np.int32)), dev(np.asarray(plan["select"][1], np.int32))]
    jk.run_draft(ctx, bufs, wts, us, root, finalize=False,
                 static_plan={"select": bad_sel, "keep": None})
    assert ctx.read_status() == jk.ERR["BOUNDS"]
    keep = np.asarray(plan["keep"], np.int32)
    keep[[2, 3]] = keep[[3, 2]]                               # not ascending
    jk.run_draft(ctx, bufs, wts, us, root,
                 static_plan={"select": [dev(np.asarray(s, np.int32)) for s in plan["select"]],
                              "keep": dev(keep)})
    assert ctx.read_status() == jk.ERR["BOUNDS"]


# ----------------------------------------------------------------- contrastive heads, hybrid schedule
@pytest.mark.parametrize("name,tensor_path", [("tiny", None), ("tiny_bf16", False),
                                              ("tiny_bf16", True)])
@pytest.mark.parametrize("residual", [True, False])
def test_contrastive_hybrid_draft(name, tensor_path, residual):
    alpha, beta = 0.35, 1.25
    w = synth.scaled(synth.WORKLOADS[name], batch=2, head_mode=1, depth=4, k_per_expert=2,
                     width=4, tree_size=16, seed=777)
    fs = w.frontier_sizes
    assert fs == [1, 2, 4] and w.n_passes == 3               # depth 4 from three passes
    ctx, bufs, wts_np, us_np = _draft(
        w, dict(contrast_alpha=alpha, contrast_beta=beta, branch_residual=residual), fs,
        tensor_path=tensor_path)
    tol = TOL[w.dtype]
    K, ke = 2, w.k_per_expert
    pool = {k: host(v) for k, v in bufs.pool.items()}
    logits = host(bufs.logits)
    gidx_base, slot_base = 0, 0
    for l, F in enumerate(fs):
        last = l == len(fs) - 1
        u = us_np[l].astype(np.float64)
        pscore = host(bufs.parent_score[l]).astype(np.float64)
        pgidx = host(bufs.parent_gidx[l])
        out = orc.draft_expand_contrastive(u, pscore, wts_np, ke, w.width, alpha, beta, last,
                                           branch_residual=residual)
        assert rel_err(host(bufs.probs[l]), out["probs"]) <= tol
        n_cand = F * K * ke
        for b in range(w.batch):
            for f in range(F):
                ids_r, _ = orc.topk_gate(host(bufs.probs[l])[b, f], K)
                assert host(bufs.expert[l])[b, f].tolist() == ids_r.tolist()
                if ids_r.tolist() == out["expert"][b, f].tolist():
                    assert rel_err(host(bufs.feat[l])[b, f], out["feat"][b, f]) <= tol
                    assert rel_err(logits[b, slot_base + f], out["logits"][b, f]) <= tol
                lg = logits[b, slot_base + f]
                g0 = gidx_base + f * K * ke
                # row 0: the node's children
                ids0, sc0, _ = orc.branch_topk(lg[0], ke, pscore[b, f])
                assert pool["tok"][b, g0:g0 + ke].tolist() == ids0.tolist()
                assert np.allclose(pool["score"][b, g0:g0 + ke], sc0, rtol=1e-5, atol=2e-5)
                assert np.all(pool["parent"][b, g0:g0 + ke] == pgidx[b, f])
                assert np.all(pool["branch"][b, g0:g0 + ke] == 0)
                # row 1: one level lower, under the best row-0 child, in the last pass only
                ids1, sc1, _ = orc.branch_topk(lg[1], ke, float(pool["score"][b, g0]))
                assert pool["tok"][b, g0 + ke:g0 + 2 * ke].tolist() == ids1.tolist()
                assert np.all(pool["parent"][b, g0 + ke:g0 + 2 * ke] == g0)
                assert np.all(pool["branch"][b, g0 + ke:g0 + 2 * ke] == 1)
                if last:
                    assert np.allclose(pool["score"][b, g0 + ke:g0 + 2 * ke], sc1, rtol=1e-5, atol=2e-5)
                else:
                    assert np.all(pool["score"][b, g0 + ke:g0 + 2 * ke] == -np.inf)
            if not last:
                sc = pool["score"][b, gidx_base:gidx_base + n_cand].reshape(F, K, ke).copy()
                sc[:, 1, :] = -np.inf                          # only row-0 children are expanded
                sel = orc.frontier_select(sc.reshape(-1), fs[l + 1])
                assert host(bufs.frontier[l])[b].tolist() == sel.tolist()
                assert host(bufs.parent_gidx[l + 1])[b].tolist() == (gidx_base + sel).tolist()
        gidx_base += n_cand
        slot_base += F
    for b in range(w.batch):
        t = orc.tree_finalize(pool["tok"][b], pool["score"][b], pool["parent"][b], pool["qslot"][b],
                              5, w.tree_size, pool_branch=pool["branch"][b])
        for key in ("tok", "parent", "depth", "branch", "qslot"):
            assert host(bufs.tree[key])[b].tolist() == t[key].tolist(), key
        assert t["depth"].max() == w.depth                     # the parallel-decoded level is there
    # greedy acceptance walks into the parallel-decoded level when the target agrees
    tree_np = {k: host(v) for k, v in bufs.tree.items()}
    tl = synth.target_logits(w, tree_np["tok"], tree_np["parent"], 1.0)
    i32 = dict(dtype=torch.int32, device="cuda")
    kvl = torch.full((w.batch,), 7, **i32)
    ctx.accept_and_compact(w.batch, w.tree_size, 0, 0.0, dev(tl), bufs.tree, None, 0, None, None, 0,
                           None, None, 0, 0, w.kv_capacity, kvl, bufs.n_acc, bufs.acc_idx,
                           bufs.acc_tok, bufs.bonus)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    for b in range(w.batch):
        path, toks, bo = orc.accept_greedy(tl[b], tree_np["tok"][b], tree_np["parent"][b])
        n = int(host(bufs.n_acc)[b])
        assert host(bufs.acc_idx)[b, :n].tolist() == path and int(host(bufs.bonus)[b]) == bo
