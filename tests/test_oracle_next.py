"""Pins of the oracle's later functions: the static tree policy (Sec. 3.1.2, last paragraph), the
contrastive head with hybrid parallel decoding (Sec. 3.2, Eq. 6-8) and the draft layer's
pre-MoE block (Eq. 1).  CPU only."""
import itertools
import math

import numpy as np
import pytest

from oracle import jakiro_oracle as orc


def _weights(rng, N=4, H=16, I=12, V=29):
    return {"router": rng.standard_normal((N, H)), "w_gate": rng.standard_normal((N, I, H)) * 0.3,
            "w_up": rng.standard_normal((N, I, H)) * 0.3, "w_down": rng.standard_normal((N, H, I)) * 0.3,
            "lm_head": rng.standard_normal((V, H)), "norm_weight": np.ones(H)}


# ----------------------------------------------------------------- static tree
PATHS = [(0,), (1,), (2,), (0, 0), (0, 2), (2, 1), (0, 0, 3), (0, 0, 0), (2, 1, 1)]


def _u_table(rng, paths, H):
    table = {(): rng.standard_normal(H)}
    for p in paths:
        table[tuple(p)] = rng.standard_normal(H)
    return table


def test_static_tree_shape_never_depends_on_the_draft():
    shapes = []
    for seed in (1, 2):
        rng = np.random.default_rng(seed)
        w = _weights(rng)
        tab = _u_table(rng, PATHS, 16)
        t = orc.grow_static_tree(lambda p: tab[p], w, PATHS, k_e=2, root_tok=3)
        shapes.append((t["parent"].tolist(), t["depth"].tolist(), t["branch"].tolist()))
        assert len(t["tok"]) == len(PATHS) + 1 and t["tok"][0] == 3
        # the parent structure is the prefix structure of the paths
        for i, p in enumerate(t["order"]):
            if p:
                assert t["order"][t["parent"][i]] == p[:-1]
                assert t["depth"][i] == len(p) and t["branch"][i] == p[-1] // 2
        assert all(t["parent"][i] < i for i in range(1, len(t["tok"])))
        assert np.all(np.diff(t["depth"]) >= 0)
    assert shapes[0] == shapes[1]


def test_static_chain_follows_the_left_experts_best_token_with_path_sum_scores():
    rng = np.random.default_rng(3)
    w = _weights(rng)
    paths = [(0,), (0, 0), (0, 0, 0)]
    tab = _u_table(rng, paths, 16)
    t = orc.grow_static_tree(lambda p: tab[p], w, paths, k_e=3, root_tok=0)
    sc = 0.0
    for i, p in enumerate(paths, start=1):
        row = t["logits"][p[:-1]][0]                      # the parent's left-branch logits
        assert t["tok"][i] == int(np.argmax(row))
        sc += row.max() - math.log(np.exp(row).sum())
        assert t["score"][i] == pytest.approx(sc, abs=1e-10)


def test_static_policy_given_the_dynamic_trees_own_shape_rebuilds_that_tree():
    # grow a dynamic tree, read its shape off as rank paths, and hand that shape to the static
    # policy with the same hidden states: the two must agree node for node
    rng = np.random.default_rng(4)
    H, k_e, width, D, M = 16, 2, 3, 3, 9
    w = _weights(rng, H=H)
    fs = [1, 3, 3]
    us = [rng.standard_normal((1, F, H)) for F in fs]
    pool = orc.grow_tree(us, w, k_e, width)
    t = orc.tree_finalize(pool["tok"][0], pool["score"][0], pool["parent"][0], pool["qslot"][0],
                          root_tok=5, tree_size=M, frontier_sizes=fs, top_k=2, k_e=k_e)
    # generation index -> (layer, frontier row, rank among the row's 2*k_e candidates)
    bases = np.cumsum([0] + [F * 2 * k_e for F in fs])
    def locate(g):
        l = int(np.searchsorted(bases, g, side="right") - 1)
        return l, (g - bases[l]) // (2 * k_e), (g - bases[l]) % (2 * k_e)
    path_of = {-1: ()}
    for g in range(pool["tok"].shape[1]):
        l, f, c = locate(g)
        path_of[g] = path_of[int(pool["parent"][0, g])] + (int(c),)
    u_of = {(): us[0][0, 0]}
    for g in range(pool["tok"].shape[1]):
        s = int(pool["qslot"][0, g])
        if s >= 0:                                         # expanded: slot -> (layer, row)
            l = int(np.searchsorted(np.cumsum([0] + fs), s, side="right") - 1)
            u_of[path_of[g]] = us[l][0, s - sum(fs[:l])]
    paths = [path_of[int(g)] for g in t["keep"]]
    st = orc.grow_static_tree(lambda p: u_of[p], w, paths, k_e, root_tok=5)
    got = {p: (int(st["tok"][i]), float(st["score"][i])) for i, p in enumerate(st["order"])}
    want = {path_of[int(g)]: (int(pool["tok"][0, g]), float(pool["score"][0, g])) for g in t["keep"]}
    want[()] = (5, 0.0)
    assert set(got) == set(want)
    for p in want:
        assert got[p][0] == want[p][0] and got[p][1] == pytest.approx(want[p][1], abs=1e-10)


def test_static_tree_rejects_orphans_and_ranks_outside_the_candidate_list():
    rng = np.random.default_rng(5)
    w = _weights(rng)
    with pytest.raises(ValueError):
        orc.grow_static_tree(lambda p: np.zeros(16), w, [(0,), (1, 0)], k_e=2, root_tok=0)
    with pytest.raises(ValueError):
        orc.grow_static_tree(lambda p: np.zeros(16), w, [(4,)], k_e=2, root_tok=0)


# ----------------------------------------------------------------- contrastive head (Eq. 6-8)
def test_contrastive_features_special_cases():
    rng = np.random.default_rng(6)
    y = rng.standard_normal((2, 10))
    g = np.array([0.6, 0.3])
    f_moe, f_const = orc.contrastive_features(y, g, alpha=0.25, beta=1.5)
    assert np.allclose(f_moe, 0.6 * y[0] + 0.3 * y[1], atol=1e-15)          # Eq. 6
    assert np.allclose(f_const, 1.5 * y[0] - 0.25 * y[1], atol=1e-15)       # Eq. 7
    # beta = s1, alpha = -s2: the contrast collapses onto the mixture
    a, b = orc.contrastive_features(y, g, alpha=-0.3, beta=0.6)
    assert np.allclose(a, b, atol=1e-15)
    # alpha = 0, beta = 1: the first expert alone
    _, c = orc.contrastive_features(y, g, alpha=0.0, beta=1.0)
    assert np.array_equal(c, y[0])
    # a sign error on alpha would show: with y1 = y2 and beta = alpha the contrast vanishes
    _, z = orc.contrastive_features(np.stack([y[0], y[0]]), g, alpha=0.7, beta=0.7)
    assert np.allclose(z, 0.0, atol=1e-15)


def test_contrastive_pass_row0_is_the_head_of_eq3_and_row1_follows_eq7():
    rng = np.random.default_rng(7)
    w = _weights(rng)
    u = rng.standard_normal((2, 3, 16))
    ps = -rng.random((2, 3))
    out = orc.draft_expand_contrastive(u, ps, w, k_e=2, width=4, alpha=0.4, beta=1.2, last_pass=True)
    ref = orc.draft_expand(u, ps, w, 2, 4)
    assert np.array_equal(out["expert"], ref["expert"])
    for b, f in itertools.product(range(2), range(3)):
        # f^moe + u is the combined feature of Eq. 3, so row 0 is its head
        assert np.allclose(out["logits"][b, f, 0], orc.head_logits(ref["feat"][b, f], w["lm_head"]),
                           atol=1e-10)
        x = orc.rmsnorm(u[b, f], w["norm_weight"], 1e-5)
        y, _, _ = orc.moe_features(u[b, f], x, ref["expert"][b, f], ref["gate"][b, f], w)
        want = orc.head_logits(1.2 * y[0] - 0.4 * y[1] + u[b, f], w["lm_head"])
        assert np.allclose(out["logits"][b, f, 1], want, atol=1e-10)
        # row-1 proposals sit under the best row-0 child: score = its score + their log-prob
        row = out["logits"][b, f, 1]
        lp = row[out["tok"][b, f, 1]] - math.log(np.exp(row).sum())
        assert np.allclose(out["score"][b, f, 1], out["score"][b, f, 0, 0] + lp, atol=1e-10)
    # without the residual the head sees Eq. 6 and Eq. 7 literally
    lit = orc.draft_expand_contrastive(u, ps, w, 2, 4, 0.4, 1.2, True, branch_residual=False)
    x = orc.rmsnorm(u[0, 0], w["norm_weight"], 1e-5)
    y, _, _ = orc.moe_features(u[0, 0], x, ref["expert"][0, 0], ref["gate"][0, 0], w)
    fm, fc = orc.contrastive_features(y, ref["gate"][0, 0], 0.4, 1.2)
    assert np.allclose(lit["logits"][0, 0], orc.head_logits(np.stack([fm, fc]), w["lm_head"]), atol=1e-10)


def test_contrastive_rows_coincide_when_the_contrast_equals_the_mixture():
    # two identical experts with equal centroids: s = (1/2, 1/2); beta = 1/2, alpha = -1/2
    rng = np.random.default_rng(8)
    w = _weights(rng, N=2)
    for k in ("router", "w_gate", "w_up", "w_down"):
        w[k][1] = w[k][0]
    u = rng.standard_normal((1, 2, 16))
    out = orc.draft_expand_contrastive(u, np.zeros((1, 2)), w, 3, 4, alpha=-0.5, beta=0.5,
                                       last_pass=True)
    assert np.allclose(out["gate"], 0.5)
    assert np.allclose(out["logits"][:, :, 0], out["logits"][:, :, 1], atol=1e-10)


def test_hybrid_schedule_reaches_depth_d_with_d_minus_one_passes():
    rng = np.random.default_rng(9)
    H, k_e, width = 16, 2, 3
    w = _weights(rng, H=H)
    fs = [1, 2, 3]                                         # 3 passes -> depth up to 4
    us = [rng.standard_normal((1, F, H)) for F in fs]
    pool = orc.grow_tree_hybrid(us, w, k_e, width, alpha=0.3, beta=1.1)
    n = pool["tok"].shape[1]
    assert n == sum(F * 2 * k_e for F in fs)
    bases = np.cumsum([0] + [F * 2 * k_e for F in fs])
    depth = {}
    for g in range(n):
        pg = int(pool["parent"][0, g])
        assert pg < g
        depth[g] = 1 if pg < 0 else depth[pg] + 1
        l = int(np.searchsorted(bases, g, side="right") - 1)
        if pool["branch"][0, g] == 1:
            # a row-1 candidate hangs under its node's best row-0 child
            f = (g - bases[l]) // (2 * k_e)
            assert pg == bases[l] + f * 2 * k_e
            assert pool["qslot"][0, g] == -1              # never expanded
            if l < len(fs) - 1:
                assert pool["score"][0, g] == -np.inf     # counts in the last pass only
            else:
                assert np.isfinite(pool["score"][0, g])
                assert pool["score"][0, g] <= pool["score"][0, pg]
    assert max(depth[g] for g in range(n) if np.isfinite(pool["score"][0, g])) == len(fs) + 1
    # expanded nodes are row-0 children only
    for g in range(n):
        if pool["qslot"][0, g] >= 0:
            assert pool["branch"][0, g] == 0
    t = orc.tree_finalize(pool["tok"][0], pool["score"][0], pool["parent"][0], pool["qslot"][0], 1,
                          12, pool_branch=pool["branch"][0])
    assert t["depth"].max() <= len(fs) + 1 and np.all(np.isfinite(t["score"]))
    assert all(t["parent"][i] < i for i in range(1, 12))


# ----------------------------------------------------------------- rotary positions
def test_rope_closed_form_norm_and_relative_property():
    x = np.array([3.0, -1.0, 0.5, 2.0])                   # d = 4: pairs (x0, x2) and (x1, x3)
    pos, theta = 7.0, 100.0
    a0, a1 = pos / theta ** 0.0, pos / theta ** 0.5
    want = [3.0 * math.cos(a0) - 0.5 * math.sin(a0), -1.0 * math.cos(a1) - 2.0 * math.sin(a1),
            0.5 * math.cos(a0) + 3.0 * math.sin(a0), 2.0 * math.cos(a1) + (-1.0) * math.sin(a1)]
    assert np.allclose(orc.rope(x, pos, theta), want, atol=1e-14)
    assert np.array_equal(orc.rope(x, 0.0, theta), x)
    rng = np.random.default_rng(10)
    q, k = rng.standard_normal(8), rng.standard_normal(8)
    assert np.linalg.norm(orc.rope(q, 13.0, 10000.0)) == pytest.approx(np.linalg.norm(q), rel=1e-13)
    d1 = orc.rope(q, 9.0, 10000.0) @ orc.rope(k, 4.0, 10000.0)
    d2 = orc.rope(q, 25.0, 10000.0) @ orc.rope(k, 20.0, 10000.0)
    assert d1 == pytest.approx(d2, rel=1e-12)             # depends on the distance only


# ----------------------------------------------------------------- draft pre-MoE block (Eq. 1)
def _pre_weights(rng, V=31, H=12, Hq=4, Hkv=2, d=4, bias=True):
    return {"emb": rng.standard_normal((V, H)), "w_fc": rng.standard_normal((H, 2 * H)) * 0.3,
            "b_fc": rng.standard_normal(H) if bias else None,
            "w_q": rng.standard_normal((Hq * d, H)) * 0.5, "w_k": rng.standard_normal((Hkv * d, H)) * 0.5,
            "w_v": rng.standard_normal((Hkv * d, H)), "w_o": rng.standard_normal((H, Hq * d)) * 0.5}


def _pre_case(seed, bias=True):
    rng = np.random.default_rng(seed)
    Hq, Hkv, d, H, P, cap = 4, 2, 4, 12, 5, 16
    pw = _pre_weights(rng, H=H, Hq=Hq, Hkv=Hkv, d=d, bias=bias)
    kc, vc = rng.standard_normal((Hkv, cap, d)), rng.standard_normal((Hkv, cap, d))
    # slots: 0 root; 1, 2 children of the root; 3, 4 children of 1; 5 child of 2
    slot_parent = np.array([-1, 0, 0, 1, 1, 2])
    return rng, pw, kc, vc, P, slot_parent, (Hq, Hkv, d, H)


def _run_layers(pw, kc, vc, P, slot_parent, dims, toks, feats, theta=50.0):
    """root layer (slot 0), then slots 1-2, then slots 3-5; returns u per slot and the caches."""
    Hq, Hkv, d, H = dims
    us = {}
    for slots in ([0], [1, 2], [3, 4, 5]):
        u, h, kc, vc = orc.draft_pre_block(toks[slots], feats[slots], pw, kc, vc, P, slots,
                                           slot_parent, Hq, Hkv, theta, 0.5)
        for i, s in enumerate(slots):
            us[s] = (u[i], h[i])
    return us, kc, vc


def test_pre_block_reduction_layer_against_loops_and_bias_switch():
    rng, pw, kc, vc, P, sp, dims = _pre_case(11)
    toks, feats = rng.integers(0, 31, 6), rng.standard_normal((6, 12))
    us, _, _ = _run_layers(pw, kc, vc, P, sp, dims, toks, feats)
    for s in range(6):
        for o in range(12):
            acc = pw["b_fc"][o]
            for j in range(12):
                acc += pw["w_fc"][o, j] * pw["emb"][toks[s], j]        # embedding first,
                acc += pw["w_fc"][o, 12 + j] * feats[s, j]             # then the feature
            assert us[s][1][o] == pytest.approx(acc, abs=1e-12)
    pw0 = dict(pw, b_fc=None)
    us0, _, _ = _run_layers(pw0, kc, vc, P, sp, dims, toks, feats)
    pwz = dict(pw, b_fc=np.zeros(12))
    usz, _, _ = _run_layers(pwz, kc, vc, P, sp, dims, toks, feats)
    assert all(np.array_equal(us0[s][0], usz[s][0]) for s in range(6))


def test_pre_block_attention_is_the_pinned_tree_attention_on_its_own_projections():
    rng, pw, kc, vc, P, sp, dims = _pre_case(12)
    Hq, Hkv, d, H = dims
    toks, feats = rng.integers(0, 31, 6), rng.standard_normal((6, 12))
    us, kc2, vc2 = _run_layers(pw, kc, vc, P, sp, dims, toks, feats)
    depth = [0, 1, 1, 2, 2, 2]
    q = np.zeros((1, 6, Hq, d))
    for s in range(6):
        qq = (pw["w_q"] @ us[s][1]).reshape(Hq, d)
        for hh in range(Hq):
            q[0, s, hh] = orc.rope(qq[hh], P + depth[s], 50.0)
        kk = (pw["w_k"] @ us[s][1]).reshape(Hkv, d)
        for hh in range(Hkv):
            assert np.allclose(kc2[hh, P + s], orc.rope(kk[hh], P + depth[s], 50.0), atol=1e-12)
        assert np.allclose(vc2[:, P + s], (pw["w_v"] @ us[s][1]).reshape(Hkv, d), atol=1e-12)
    att = orc.tree_verify_attn(q, kc2[None], vc2[None], np.array([P]), sp[None], 0.5)
    for s in range(6):
        want = pw["w_o"] @ att[0, s].reshape(-1) + us[s][1]                # u = Attn(h) + h
        assert np.allclose(us[s][0], want, atol=1e-10)
    # rows that belong to no node keep their contents
    live = set(range(P, P + 6))
    for r in range(kc.shape[1]):
        if r not in live:
            assert np.array_equal(kc2[:, r], kc[:, r]) and np.array_equal(vc2[:, r], vc[:, r])


def test_pre_block_node_depends_on_its_root_path_only():
    rng, pw, kc, vc, P, sp, dims = _pre_case(13, bias=False)
    toks, feats = rng.integers(0, 31, 6), rng.standard_normal((6, 12))
    us, _, _ = _run_layers(pw, kc, vc, P, sp, dims, toks, feats)
    # node 5's path is 0 -> 2 -> 5: rebuild it as a chain of three slots
    chain = [0, 2, 5]
    Hq, Hkv, d, H = dims
    kc1, vc1 = kc.copy(), vc.copy()
    u_last = None
    for i, s in enumerate(chain):
        u, h, kc1, vc1 = orc.draft_pre_block(toks[[s]], feats[[s]], pw, kc1, vc1, P, [i],
                                             np.array([-1, 0, 1]), Hq, Hkv, 50.0, 0.5)
        u_last = u[0]
    assert np.allclose(u_last, us[5][0], atol=1e-10)


def test_pre_block_uniform_attention_closed_form():
    # W_q = 0: every visible column gets the same weight, so Attn is the mean of the visible V rows
    rng, pw, kc, vc, P, sp, dims = _pre_case(14)
    Hq, Hkv, d, H = dims
    pw = dict(pw, w_q=np.zeros_like(pw["w_q"]))
    toks, feats = rng.integers(0, 31, 6), rng.standard_normal((6, 12))
    us, kc2, vc2 = _run_layers(pw, kc, vc, P, sp, dims, toks, feats)
    cols = list(range(P)) + [P + 0, P + 1, P + 4]                          # node 4: 0 -> 1 -> 4
    mean_v = vc2[:, cols].mean(axis=1)                                     # [Hkv, d]
    o = np.stack([mean_v[hh // (Hq // Hkv)] for hh in range(Hq)]).reshape(-1)
    assert np.allclose(us[4][0], pw["w_o"] @ o + us[4][1], atol=1e-10)


# ----------------------------------------------------------------- verification-side glue
def test_verify_qkv_append_against_loops_and_the_attention_it_feeds():
    rng = np.random.default_rng(20)
    M, H, Hq, Hkv, d, P, cap = 5, 6, 4, 2, 4, 3, 12
    x = rng.standard_normal((M, H))
    wq, wk, wv = (rng.standard_normal((Hq * d, H)), rng.standard_normal((Hkv * d, H)),
                  rng.standard_normal((Hkv * d, H)))
    parent = np.array([-1, 0, 0, 1, 3])
    depth = np.array([0, 1, 1, 2, 3])
    kc, vc = rng.standard_normal((Hkv, cap, d)), rng.standard_normal((Hkv, cap, d))
    q, kc2, vc2 = orc.verify_qkv_append(x, wq, wk, wv, depth, kc, vc, P, Hq, Hkv, 77.0)
    for i in range(M):
        for hh in range(Hq):
            raw = [sum(wq[hh * d + c, j] * x[i, j] for j in range(H)) for c in range(d)]
            assert np.allclose(q[i, hh], orc.rope(np.array(raw), P + depth[i], 77.0), atol=1e-12)
        for hh in range(Hkv):
            raw = [sum(wk[hh * d + c, j] * x[i, j] for j in range(H)) for c in range(d)]
            assert np.allclose(kc2[hh, P + i], orc.rope(np.array(raw), P + depth[i], 77.0), atol=1e-12)
            raw = [sum(wv[hh * d + c, j] * x[i, j] for j in range(H)) for c in range(d)]
            assert np.allclose(vc2[hh, P + i], raw, atol=1e-12)        # V is not rotated
    untouched = [r for r in range(cap) if not P <= r < P + M]
    assert np.array_equal(kc2[:, untouched], kc[:, untouched])
    # siblings (nodes 1 and 2, both depth 1) share a position: equal inputs give equal q and k
    x2 = x.copy()
    x2[2] = x2[1]
    q2, k2, _ = orc.verify_qkv_append(x2, wq, wk, wv, depth, kc, vc, P, Hq, Hkv, 77.0)
    assert np.array_equal(q2[1], q2[2]) and np.array_equal(k2[:, P + 1], k2[:, P + 2])
    # chain tree: the rows it writes are those of a plain causal decode at positions P, P+1, ...
    chain_depth = np.arange(M)
    qc, kcc, _ = orc.verify_qkv_append(x, wq, wk, wv, chain_depth, kc, vc, P, Hq, Hkv, 77.0)
    for i in range(M):
        raw = (wk @ x[i]).reshape(Hkv, d)
        assert np.allclose(kcc[0, P + i], orc.rope(raw[0], P + i, 77.0), atol=1e-12)


def test_gather_accepted_rows():
    hidden = np.arange(24.0).reshape(6, 4)
    out = orc.gather_accepted(hidden, [2, 5], rows=5)
    assert np.array_equal(out[0], hidden[0]) and np.array_equal(out[1], hidden[2])
    assert np.array_equal(out[2], hidden[5]) and np.all(out[3:] == 0)
    assert np.array_equal(orc.gather_accepted(hidden, [], rows=3)[1:], np.zeros((2, 4)))
