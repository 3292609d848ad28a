"""GPU parity of jk_draft_expand / jk_tree_finalize against the CPU oracle.

Floating stages are compared by tolerance with the oracle's own computation on the same inputs;
every discrete decision (experts, top-k tokens, frontier, final tree) is re-derived by the oracle
from the GPU's floating inputs to that decision and compared exactly.
"""
import numpy as np
import pytest
import torch

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import binding as jk
from paper_2502_06282_b200 import synth
from tests.jk_testutil import (TOL, Guard, dev, guarded_context, guarded_step_buffers, host,
                                rel_err, weights_to_device)

pytestmark = pytest.mark.gpu


def _run_gpu(w, wts_np, us_np, tensor_path=None, root_tok=5, expect_tensor_path=None, **ctx_kw):
    """One draft (D expand calls + finalize) with every output buffer and the workspace poisoned
    and fenced by canaries; the canaries are checked before the results are returned."""
    ctx, check_ws = guarded_context(w, **ctx_kw)
    if tensor_path is not None:
        ctx.set_tensor_path(tensor_path)
        assert ctx.tensor_path_active == bool(tensor_path)
    if expect_tensor_path is not None:
        assert ctx.tensor_path_active == expect_tensor_path
    guard = Guard()
    bufs = guarded_step_buffers(ctx, w, guard)
    wts = weights_to_device(wts_np, w.dtype)
    us = [dev(u, w.dtype) for u in us_np]
    root = torch.full((w.batch,), root_tok, dtype=torch.int32, device="cuda")
    jk.run_draft(ctx, bufs, wts, us, root)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    guard.check()
    check_ws()
    return ctx, bufs


def _check_layers(w, wts_np, us_np, bufs, use_pre_norm=True, branch_residual=True, rms_eps=1e-5):
    tol = TOL[w.dtype]
    fs = w.frontier_sizes
    K, ke = w.top_k, w.k_per_expert
    gidx_base, slot_base = 0, 0
    pool = {k: host(v) for k, v in bufs.pool.items()}
    logits_all = host(bufs.logits)
    for l, F in enumerate(fs):
        u = us_np[l].astype(np.float64)
        pscore = host(bufs.parent_score[l]).astype(np.float64)
        pgidx = host(bufs.parent_gidx[l])
        probs_g, exp_g, gate_g = host(bufs.probs[l]), host(bufs.expert[l]), host(bufs.gate[l])
        feat_g, lse_g = host(bufs.feat[l]), host(bufs.lse[l])
        x = orc.rmsnorm(u, wts_np["norm_weight"], rms_eps) if use_pre_norm else u
        probs_o = orc.router_scores(x, wts_np["router"])
        assert rel_err(probs_g, probs_o) <= tol
        n_cand = F * K * ke
        for b in range(w.batch):
            for f in range(F):
                # experts: replayed from the GPU's own scores, exact
                ids_r, g_r = orc.topk_gate(probs_g[b, f], K)
                assert exp_g[b, f].tolist() == ids_r.tolist()
                assert np.array_equal(gate_g[b, f], probs_g[b, f][ids_r])
                ids_o, _ = orc.topk_gate(probs_o[b, f], K)
                margin = np.sort(probs_o[b, f])[::-1]
                if margin[K - 1] - margin[K] > 1e-3 and (K < 2 or margin[0] - margin[1] > 1e-3):
                    assert ids_o.tolist() == ids_r.tolist()
                _, br, ff = orc.moe_features(u[b, f], x[b, f], ids_r, probs_o[b, f][ids_r], wts_np,
                                             branch_residual)
                assert rel_err(feat_g[b, f], ff) <= tol
                lg_o = orc.head_logits(br, wts_np["lm_head"])
                lg_g = logits_all[b, slot_base + f]
                assert rel_err(lg_g, lg_o) <= tol
                for r in range(K):
                    # top-k tokens and scores: replayed from the GPU's logits
                    ids_t, sc_t, lse_t = orc.branch_topk(lg_g[r], ke, pscore[b, f])
                    g0 = gidx_base + (f * K + r) * ke
                    assert pool["tok"][b, g0:g0 + ke].tolist() == ids_t.tolist()
                    assert np.allclose(pool["score"][b, g0:g0 + ke], sc_t, rtol=1e-5, atol=2e-5)
                    assert abs(lse_g[b, f, r] - lse_t) <= 2e-5 * max(1.0, abs(lse_t))
                    assert np.all(pool["parent"][b, g0:g0 + ke] == pgidx[b, f])
                    assert np.all(pool["branch"][b, g0:g0 + ke] == r)
            if l < len(fs) - 1:
                sel = orc.frontier_select(pool["score"][b, gidx_base:gidx_base + n_cand],
                                          min(w.width, n_cand))
                assert host(bufs.frontier[l])[b].tolist() == sel.tolist()
                assert np.array_equal(host(bufs.parent_score[l + 1])[b],
                                      pool["score"][b, gidx_base + sel])
                assert host(bufs.parent_gidx[l + 1])[b].tolist() == (gidx_base + sel).tolist()
                q = np.full(n_cand, -1)
                q[sel] = slot_base + F + np.arange(len(sel))
                assert pool["qslot"][b, gidx_base:gidx_base + n_cand].tolist() == q.tolist()
            else:
                assert np.all(pool["qslot"][b, gidx_base:gidx_base + n_cand] == -1)
        gidx_base += n_cand
        slot_base += F
    return pool


def _check_tree(w, pool, bufs, root_tok):
    for b in range(w.batch):
        t = orc.tree_finalize(pool["tok"][b], pool["score"][b], pool["parent"][b],
                              pool["qslot"][b], root_tok, w.tree_size,
                              pool_branch=pool["branch"][b])
        for key in ("tok", "parent", "depth", "branch", "qslot"):
            assert host(bufs.tree[key])[b].tolist() == t[key].tolist(), key
        anc = orc.ancestor_mask(t["parent"])
        bits = host(bufs.anc)[b].astype(np.uint64)
        for i in range(w.tree_size):
            got = [(int(bits[i, c >> 6]) >> (c & 63)) & 1 for c in range(w.tree_size)]
            assert got == anc[i].astype(int).tolist()


def _inputs(w):
    wts = synth.draft_weights(w)
    us = [synth.layer_hidden(w, l, F) for l, F in enumerate(w.frontier_sizes)]
    return wts, us


@pytest.mark.parametrize("name,tensor_path", [("tiny", None), ("tiny_bf16", False),
                                              ("tiny_bf16", True)])
def test_expand_tiny_full_parity(name, tensor_path):
    w = synth.WORKLOADS[name]
    wts, us = _inputs(w)
    ctx, bufs = _run_gpu(w, wts, us, tensor_path)
    pool = _check_layers(w, wts, us, bufs)
    _check_tree(w, pool, bufs, 5)
    if w.dtype == "f32":
        # no near-ties in this seeded case: the oracle's own tree is the same tree
        ref = orc.grow_tree(us, wts, w.k_per_expert, w.width)
        t = orc.tree_finalize(ref["tok"][0], ref["score"][0], ref["parent"][0], ref["qslot"][0],
                              5, w.tree_size, frontier_sizes=w.frontier_sizes,
                              top_k=w.top_k, k_e=w.k_per_expert)
        assert host(bufs.tree["tok"])[0].tolist() == t["tok"].tolist()
        assert host(bufs.tree["parent"])[0].tolist() == t["parent"].tolist()


@pytest.mark.parametrize("tensor_path", [False, True])
def test_expand_batched_ragged_shapes(tensor_path):
    # batch 3, vocabulary and inner size that end in partial tiles, N = 3 experts, k_e = 3
    w = synth.scaled(synth.WORKLOADS["tiny_bf16"], name="ragged", batch=3, vocab=5000,
                     inter=1000, hidden=264, n_experts=3, k_per_expert=3, width=5,
                     tree_size=20, depth=3, seed=77)
    wts, us = _inputs(w)
    ctx, bufs = _run_gpu(w, wts, us, tensor_path)
    pool = _check_layers(w, wts, us, bufs)
    _check_tree(w, pool, bufs, 5)


def test_expand_f32_ragged_shapes():
    w = synth.scaled(synth.WORKLOADS["tiny"], name="ragged32", batch=2, vocab=4100, inter=520,
                     hidden=136, n_experts=5, k_per_expert=4, width=6, tree_size=25, depth=3,
                     seed=78)
    wts, us = _inputs(w)
    ctx, bufs = _run_gpu(w, wts, us)
    pool = _check_layers(w, wts, us, bufs)
    _check_tree(w, pool, bufs, 5)


@pytest.mark.parametrize("name,tensor_path", [("tiny", None), ("tiny_bf16", False),
                                              ("tiny_bf16", True)])
@pytest.mark.parametrize("use_pre_norm,branch_residual", [(False, True), (True, False),
                                                          (False, False)])
def test_expand_config_flags(name, tensor_path, use_pre_norm, branch_residual):
    """The two readings the configuration can switch: no pre-MoE normalisation (router and
    experts see u itself), and branch features without the residual (Eq. 4 taken literally as
    Head(s_r * Expert_r)).  Hidden states three times larger than unit RMS, a norm weight that
    is not all ones and a large epsilon make each switch change the result well beyond the
    tolerance, so a flag that the kernels ignored could not pass."""
    w = synth.scaled(synth.WORKLOADS[name], batch=2, depth=3, tree_size=14, seed=4242)
    wts, us = _inputs(w)
    gamma = 0.5 + np.random.default_rng(3).random(w.hidden).astype(np.float32)
    wts["norm_weight"] = synth.store_round(gamma, w.dtype)
    us = [synth.store_round(3.0 * u, w.dtype) for u in us]
    eps = 0.75
    ctx, bufs = _run_gpu(w, wts, us, tensor_path, use_pre_norm=use_pre_norm,
                         branch_residual=branch_residual, rms_eps=eps)
    pool = _check_layers(w, wts, us, bufs, use_pre_norm, branch_residual, eps)
    _check_tree(w, pool, bufs, 5)
    # the switch matters on these inputs: the other setting is far outside the tolerance
    u0 = us[0].astype(np.float64)
    other = orc.draft_expand(u0, np.zeros((w.batch, 1)), wts, w.k_per_expert, w.width,
                             rms_eps=eps, use_pre_norm=not use_pre_norm,
                             branch_residual=branch_residual)
    assert rel_err(host(bufs.logits)[:, 0], other["logits"][:, 0]) > 10 * TOL[w.dtype]
    other = orc.draft_expand(u0, np.zeros((w.batch, 1)), wts, w.k_per_expert, w.width,
                             rms_eps=eps, use_pre_norm=use_pre_norm,
                             branch_residual=not branch_residual)
    assert rel_err(host(bufs.logits)[:, 0], other["logits"][:, 0]) > 10 * TOL[w.dtype]


@pytest.mark.parametrize("name,tensor_path", [("tiny", None), ("tiny_bf16", False),
                                              ("tiny_bf16", True)])
def test_expand_planted_ties(name, tensor_path):
    """Two vocabulary rows of the LM head made identical, chosen so that they are the root's best
    left-branch tokens: their logits are equal bit for bit (same weight tile, same summation
    order), so the top-k order and the frontier order are both decided by the tie rule (lower
    token id, then lower candidate index)."""
    w = synth.WORKLOADS[name]
    wts, us = _inputs(w)
    _, first = _run_gpu(w, wts, us, tensor_path)
    t1 = int(host(first.pool["tok"])[0, 0])
    t2 = t1 ^ 1
    wts["lm_head"] = wts["lm_head"].copy()
    wts["lm_head"][t2] = wts["lm_head"][t1]
    ctx, bufs = _run_gpu(w, wts, us, tensor_path)
    lg = host(bufs.logits)[0, 0, 0]
    assert lg[t1] == lg[t2]
    pool = _check_layers(w, wts, us, bufs)
    assert pool["tok"][0, :2].tolist() == sorted([t1, t2])
    assert pool["score"][0, 0] == pool["score"][0, 1]
    fr = host(bufs.frontier[0])[0].tolist()
    assert fr.index(0) < fr.index(1)                 # equal scores: the lower index goes first
    _check_tree(w, pool, bufs, 5)


@pytest.mark.parametrize("name,tensor_path", [("tiny", None), ("tiny_bf16", True)])
def test_expand_many_equal_logits(name, tensor_path):
    """Three hundred vocabulary rows of the LM head made identical to the root's best token: more
    entries reach the chunk's selection threshold than its short candidate list holds, so the
    full selection runs instead, and the tie rule (lower token id first) decides the top-k."""
    w = synth.WORKLOADS[name]
    assert w.vocab >= 400
    wts, us = _inputs(w)
    _, first = _run_gpu(w, wts, us, tensor_path)
    t1 = int(host(first.pool["tok"])[0, 0])
    wts["lm_head"] = wts["lm_head"].copy()
    wts["lm_head"][40:340] = wts["lm_head"][t1]
    ctx, bufs = _run_gpu(w, wts, us, tensor_path)
    lg = host(bufs.logits)[0, 0, 0]
    assert np.all(lg[40:340] == lg[t1])
    pool = _check_layers(w, wts, us, bufs)
    ke = w.k_per_expert
    want = sorted(set(range(40, 340)) | {t1})[:ke]
    assert pool["tok"][0, :ke].tolist() == want
    _check_tree(w, pool, bufs, 5)


def test_expand_tensor_path_row_limit_and_fallback():
    """128 activation rows with K = 2 give 256 logits rows, the most the tensor-core GEMM takes
    (two accumulators of 256 columns fill the tensor memory); with K = 3 the same rows give 384,
    the context reports the tensor path as inactive and the CUDA-core kernels run instead."""
    base = dict(name="rows", batch=8, hidden=256, inter=512, vocab=4096, depth=2, tree_size=24,
                width=16, seed=91)
    w = synth.scaled(synth.WORKLOADS["tiny_bf16"], k_per_expert=8, **base)
    assert w.frontier_sizes == [1, 16]
    wts, us = _inputs(w)
    ctx, bufs = _run_gpu(w, wts, us, expect_tensor_path=True)
    pool = _check_layers(w, wts, us, bufs)
    _check_tree(w, pool, bufs, 5)
    w3 = synth.scaled(synth.WORKLOADS["tiny_bf16"], k_per_expert=6, top_k=3, **base)
    assert w3.frontier_sizes == [1, 16]
    wts, us = _inputs(w3)
    ctx, bufs = _run_gpu(w3, wts, us, expect_tensor_path=False)
    pool = _check_layers(w3, wts, us, bufs)
    _check_tree(w3, pool, bufs, 5)


def test_expand_is_deterministic():
    w = synth.WORKLOADS["tiny_bf16"]
    wts, us = _inputs(w)
    _, a = _run_gpu(w, wts, us)
    _, b = _run_gpu(w, wts, us)
    assert torch.equal(a.logits, b.logits)
    for k in a.pool:
        assert torch.equal(a.pool[k], b.pool[k])


def _sampled_rows(w, samples, wts=None, wts_dev=None):
    """len(samples) draft layers at full-size shapes, launch configuration as benchmarked; the
    oracle recomputes the (batch, frontier row) pairs in `samples[layer]`.  `wts` may hold
    per-expert matrices behind lazy sequences (and `wts_dev` the device copies made expert by
    expert) for shapes whose full fp32 weight set would not fit the host."""
    if wts is None:
        wts = synth.draft_weights(w)
    n_l = len(samples)
    fs = w.frontier_sizes[:n_l]
    us = [synth.layer_hidden(w, l, F) for l, F in enumerate(fs)]
    w2 = synth.scaled(w, depth=n_l, tree_size=min(w.tree_size, 12))
    ctx, check_ws = guarded_context(w2)
    guard = Guard()
    bufs = guarded_step_buffers(ctx, w2, guard)
    if wts_dev is None:
        wts_dev = weights_to_device(wts, w.dtype)
    root = torch.full((w.batch,), 5, dtype=torch.int32, device="cuda")
    jk.run_draft(ctx, bufs, wts_dev, [dev(u, w.dtype) for u in us], root)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    guard.check()
    check_ws()
    tol = TOL[w.dtype]
    head64 = np.asarray(wts["lm_head"], dtype=np.float64)
    K, ke = w.top_k, w.k_per_expert
    slot_base, gidx_base = 0, 0
    pool_tok, pool_score = host(bufs.pool["tok"]), host(bufs.pool["score"])
    for l, F in enumerate(fs):
        u = us[l].astype(np.float64)
        probs_g = host(bufs.probs[l])
        pscore = host(bufs.parent_score[l])
        for b, f in samples[l]:
            x = orc.rmsnorm(u[b, f], wts["norm_weight"], 1e-5)
            probs_o = orc.router_scores(x, wts["router"])
            assert rel_err(probs_g[b, f], probs_o) <= tol
            ids, _ = orc.topk_gate(probs_g[b, f], K)
            assert host(bufs.expert[l])[b, f].tolist() == ids.tolist()
            _, br, ff = orc.moe_features(u[b, f], x, ids, probs_o[ids], wts)
            assert rel_err(host(bufs.feat[l])[b, f], ff) <= tol
            lg_o = br @ head64.T
            lg_g = host(bufs.logits[b, slot_base + f])
            assert rel_err(lg_g, lg_o) <= tol
            for r in range(K):
                ids_t, sc_t, _ = orc.branch_topk(lg_g[r], ke, float(pscore[b, f]))
                g0 = gidx_base + (f * K + r) * ke
                assert pool_tok[b, g0:g0 + ke].tolist() == ids_t.tolist()
                assert np.allclose(pool_score[b, g0:g0 + ke], sc_t, rtol=1e-5, atol=2e-5)
        # the frontier of every layer but the last, replayed from the GPU's scores
        n_cand = F * K * ke
        if l < n_l - 1:
            for b in range(w.batch):
                sel = orc.frontier_select(pool_score[b, gidx_base:gidx_base + n_cand],
                                          min(w.width, n_cand))
                assert host(bufs.frontier[l])[b].tolist() == sel.tolist()
                assert host(bufs.parent_gidx[l + 1])[b].tolist() == (gidx_base + sel).tolist()
        slot_base += F
        gidx_base += n_cand
    return bufs


def test_expand_llama2_7b_shape_sampled_rows():
    _sampled_rows(synth.WORKLOADS["llama2_7b"], [[(0, 0)], [(0, 3), (0, 8)]])


def test_expand_llama2_7b_shape_all_layers():
    """All six draft layers of the benchmarked step (frontier sizes 1, 10, 10, 10, 10, 10): the
    pool offsets, slot offsets and per-sequence logits stride of the deeper layers, one or two
    sampled rows per layer."""
    w = synth.WORKLOADS["llama2_7b"]
    assert w.frontier_sizes == [1, 10, 10, 10, 10, 10]
    bufs = _sampled_rows(w, [[(0, 0)], [(0, 9)], [(0, 2)], [(0, 0), (0, 7)], [(0, 5)], [(0, 9)]])
    pool = {k: host(v) for k, v in bufs.pool.items()}
    t = orc.tree_finalize(pool["tok"][0], pool["score"][0], pool["parent"][0], pool["qslot"][0],
                          5, 12, pool_branch=pool["branch"][0])
    for key in ("tok", "parent", "depth", "branch", "qslot"):
        assert host(bufs.tree[key])[0].tolist() == t[key].tolist(), key


def test_expand_llama2_13b_batch4_sampled_rows():
    # 4 sequences x 10 frontier rows = 40 activation rows (48 after padding), 80 logits rows
    _sampled_rows(synth.WORKLOADS["llama2_13b_b4"], [[(2, 0)], [(0, 9), (3, 4)]])


def test_expand_llama3_8b_vocab_sampled_rows():
    # vocabulary 128256: 32 top-k chunks per row, LM head dominates the bytes
    _sampled_rows(synth.WORKLOADS["llama3_8b"], [[(0, 0)], [(0, 6)]])


def test_expand_llama2_70b_shape_two_experts():
    # hidden 8192, inner 28672; N = K = 2 (the setting with the best speedup in Table 3) keeps
    # the host-side weight generation of this test affordable
    w = synth.scaled(synth.WORKLOADS["llama2_70b_layer"], n_experts=2, name="llama2_70b_n2")
    _sampled_rows(w, [[(0, 0)], [(0, 5)]])


class _LazyExperts:
    """w_gate / w_up / w_down of a workload whose experts are drawn one at a time."""

    def __init__(self, w, name):
        self.w, self.name = w, name

    def __getitem__(self, e):
        return synth.expert_weight(self.w, self.name, int(e))


def test_expand_llama2_70b_shape_four_experts():
    """The 70B layer shape as configured (N = 4, hidden 8192, inner 28672): 5.6 GB of bf16 expert
    weights on the device.  The host never holds more than one expert matrix in fp32: device
    tensors are filled expert by expert and the oracle draws the experts it needs again."""
    w = synth.WORKLOADS["llama2_70b_layer"]
    assert w.n_experts == 4 and w.inter == 28672
    small = synth.shared_weights(w)
    wts = dict(small)
    wts_dev = {k: dev(v, w.dtype) for k, v in small.items()}
    for name, shape in (("w_gate", (w.inter, w.hidden)), ("w_up", (w.inter, w.hidden)),
                        ("w_down", (w.hidden, w.inter))):
        t = torch.empty((w.n_experts,) + shape, dtype=torch.bfloat16, device="cuda")
        for e in range(w.n_experts):
            t[e].copy_(dev(synth.expert_weight(w, name, e), w.dtype))
        wts_dev[name] = t
        wts[name] = _LazyExperts(w, name)
    _sampled_rows(w, [[(0, 0)], [(0, 4)]], wts=wts, wts_dev=wts_dev)


# ------------------------------------------------------------ jk_tree_finalize on hand-made pools
def _made_pool(rng, fs, K, ke, levels=None):
    """A pool with the structure the draft produces (parents before children, a child never above
    its parent, the next frontier = the best of a layer), scores in fp32.  `levels`: quantise the
    increments to that many values, which makes many scores equal."""
    tok, score, parent, qslot, branch = [], [], [], [], []
    frontier = [(-1, np.float32(0.0))]
    slot = 1
    for l, F in enumerate(fs):
        assert len(frontier) == F
        first = len(tok)
        for pg, ps in frontier:
            for r in range(K):
                inc = np.sort(rng.exponential(1.0, ke))
                if levels:
                    inc = np.ceil(inc * levels) / levels
                for j in range(ke):
                    tok.append(int(rng.integers(0, 64)))
                    score.append(np.float32(ps - np.float32(inc[j])))
                    parent.append(pg)
                    qslot.append(-1)
                    branch.append(r)
        if l + 1 < len(fs):
            layer = np.asarray(score[first:], np.float32)
            sel = orc.frontier_select(layer, fs[l + 1])
            frontier = []
            for s_ in sel:
                qslot[first + int(s_)] = slot
                slot += 1
                frontier.append((first + int(s_), layer[int(s_)]))
    return {"tok": np.asarray(tok, np.int32), "score": np.asarray(score, np.float32),
            "parent": np.asarray(parent, np.int32), "qslot": np.asarray(qslot, np.int32),
            "branch": np.asarray(branch, np.int32)}


@pytest.mark.parametrize("fs,ke,M,levels", [
    ([1, 10, 10, 10, 10, 10], 5, 60, None),      # 510 candidates: the bound cuts the pool down
    ([1, 10, 10, 10, 10, 10], 5, 60, 2),         # many equal scores: more reach the bound than fit
    ([1, 10, 10, 10, 10, 10], 5, 128, None),     # 127 kept of 510
    ([1, 10, 20, 20, 20, 20], 5, 100, None),     # 910 candidates in 114 runs of 8, 99 kept
    ([1, 10, 20, 20, 20, 20], 5, 128, None),     # the same pool, 127 kept: ranked whole
    ([1, 12, 12], 6, 100, None),                 # 300 candidates in runs of 3: 100 runs for 99 kept
    ([1, 6, 6, 6], 5, 40, None),                 # 190 candidates: ranked whole
    ([1, 5, 5], 13, 128, None),                  # 286 candidates in 96 runs, 127 kept: ranked whole
])
def test_tree_finalize_made_pools(fs, ke, M, levels):
    K, B = 2, 3
    rng = np.random.default_rng(len(fs) * 1000 + ke * 10 + M)
    pools = [_made_pool(rng, fs, K, ke, levels) for _ in range(B)]
    pool_n = len(pools[0]["tok"])
    w = synth.scaled(synth.WORKLOADS["tiny"], batch=B, tree_size=M, k_per_expert=ke,
                     depth=len(fs), width=max(fs))
    ctx = jk.Context.for_workload(w, frontier_sizes=fs)
    pool = {k: dev(np.stack([p[k] for p in pools])) for k in pools[0]}
    i32 = dict(dtype=torch.int32, device="cuda")
    tree = {k: torch.full((B, M), -7, **i32) for k in ("tok", "parent", "depth", "branch", "qslot")}
    anc = torch.zeros(B, M, 2, dtype=torch.int64, device="cuda")
    root = torch.arange(5, 5 + B, **i32)
    ctx.tree_finalize(B, pool, pool_n, root, M, tree["tok"], tree["parent"], tree["depth"],
                      tree["branch"], tree["qslot"], anc)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    for b in range(B):
        p = pools[b]
        t = orc.tree_finalize(p["tok"], p["score"], p["parent"], p["qslot"], 5 + b, M,
                              pool_branch=p["branch"])
        for key in ("tok", "parent", "depth", "branch", "qslot"):
            assert host(tree[key])[b].tolist() == t[key].tolist(), (b, key)
        am = orc.ancestor_mask(t["parent"])
        bits = host(anc)[b].astype(np.uint64)
        for i in range(M):
            got = [(int(bits[i, c // 64]) >> (c % 64)) & 1 for c in range(M)]
            assert got == am[i].astype(int).tolist()
