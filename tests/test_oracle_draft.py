"""Pins for the oracle's draft layer (router, experts, head, top-k, tree growth).

Each test ties one oracle function to something outside it: a closed form, a
pure-Python brute force, or an invariant the paper states (Sec. 3.1.2, Eq. 2-5).
"""
import itertools
import math

import numpy as np
import pytest

from oracle import jakiro_oracle as orc


def _weights(rng, N, H, I, V, std=0.3):
    return {
        "router": rng.standard_normal((N, H)) * std,
        "w_gate": rng.standard_normal((N, I, H)) * std,
        "w_up": rng.standard_normal((N, I, H)) * std,
        "w_down": rng.standard_normal((N, H, I)) * std,
        "lm_head": rng.standard_normal((V, H)) * std,
        "norm_weight": np.ones(H),
    }


# ----------------------------------------------------------------- router (Eq. 2, Eq. 5)
def test_router_two_experts_is_a_sigmoid():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 7))
    E = rng.standard_normal((2, 7))
    s = orc.router_scores(x, E)
    for i in range(5):
        z0 = sum(x[i, k] * E[0, k] for k in range(7))
        z1 = sum(x[i, k] * E[1, k] for k in range(7))
        assert s[i, 0] == pytest.approx(1.0 / (1.0 + math.exp(z1 - z0)), rel=1e-12)
        assert s[i, 0] + s[i, 1] == pytest.approx(1.0, abs=1e-14)


def test_router_rows_sum_to_one_and_are_shift_invariant():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((4, 9))
    E = rng.standard_normal((5, 9))
    s = orc.router_scores(x, E)
    assert np.allclose(s.sum(-1), 1.0, atol=1e-14)
    # adding the same vector to every centroid shifts all N logits equally
    s2 = orc.router_scores(x, E + rng.standard_normal((1, 9)))
    assert np.allclose(s, s2, atol=1e-12)


def test_gate_keeps_exactly_k_scores_unrenormalised_left_is_larger():
    s = np.array([0.1, 0.4, 0.2, 0.3])
    ids, g = orc.topk_gate(s, 2)
    assert ids.tolist() == [1, 3]            # left = larger score
    assert g.tolist() == [0.4, 0.3]          # the scores themselves (Eq. 5)
    dense = np.zeros(4)
    dense[ids] = g
    assert np.count_nonzero(dense) == 2


def test_gate_ties_go_to_lower_expert_id_and_n_equals_k_selects_all():
    ids, g = orc.topk_gate(np.array([0.25, 0.25, 0.25, 0.25]), 2)
    assert ids.tolist() == [0, 1]
    ids, g = orc.topk_gate(np.array([0.3, 0.7]), 2)       # N = K = 2 (Table 3, best speedup)
    assert ids.tolist() == [1, 0] and g.tolist() == [0.7, 0.3]


def test_rmsnorm_unit_rms():
    rng = np.random.default_rng(3)
    u = rng.standard_normal((3, 64)) * 5
    x = orc.rmsnorm(u, None, 0.0)
    assert np.allclose(np.sqrt((x * x).mean(-1)), 1.0, atol=1e-12)
    x2 = orc.rmsnorm(u * 7.0, None, 0.0)
    assert np.allclose(x, x2, atol=1e-12)    # scale invariance
    g = rng.standard_normal(64)
    assert np.allclose(orc.rmsnorm(u, g, 0.0), x * g, atol=1e-12)


def test_rmsnorm_epsilon_sits_inside_the_square_root():
    # constant row c: mean square = c^2, so x = c / sqrt(c^2 + eps) in closed form.  With
    # c = 3, eps = 16 that is 3/5; an epsilon added outside the root would give 3/19, an
    # epsilon ignored 1, an epsilon on the sum instead of the mean 3/sqrt(9 + 16/H).
    x = orc.rmsnorm(np.full((2, 8), 3.0), None, 16.0)
    assert np.allclose(x, 0.6, atol=1e-15)
    x = orc.rmsnorm(np.full((1, 4), -3.0), np.array([1.0, 2.0, -1.0, 0.5]), 16.0)
    assert np.allclose(x, [[-0.6, -1.2, 0.6, -0.3]], atol=1e-15)
    # a zero row stays zero instead of dividing by zero
    assert np.all(orc.rmsnorm(np.zeros((1, 4)), None, 1e-5) == 0.0)


# ----------------------------------------------------------------- experts (Eq. 3)
def test_expert_ffn_against_pure_python_loops():
    rng = np.random.default_rng(4)
    H, I = 6, 5
    x = rng.standard_normal(H)
    Wg, Wu, Wd = rng.standard_normal((I, H)), rng.standard_normal((I, H)), rng.standard_normal((H, I))
    y = orc.expert_ffn(x, Wg, Wu, Wd)
    for o in range(H):
        acc = 0.0
        for i in range(I):
            g = sum(Wg[i, k] * x[k] for k in range(H))
            a = sum(Wu[i, k] * x[k] for k in range(H))
            acc += Wd[o, i] * (g / (1.0 + math.exp(-g))) * a
        assert y[o] == pytest.approx(acc, rel=1e-11, abs=1e-12)


def test_expert_transposed_operand_would_fail():
    # W_gate and W_up are [I, H], W_down is [H, I]: a non-square case has only one
    # consistent reading, and a zero W_up row kills exactly that inner unit
    rng = np.random.default_rng(5)
    H, I = 4, 7
    x = rng.standard_normal(H)
    Wg, Wu, Wd = rng.standard_normal((I, H)), rng.standard_normal((I, H)), rng.standard_normal((H, I))
    y0 = orc.expert_ffn(x, Wg, Wu, Wd)
    Wu2 = Wu.copy(); Wu2[3] = 0.0
    Wd2 = Wd.copy(); Wd2[:, 3] = 0.0
    assert np.allclose(orc.expert_ffn(x, Wg, Wu2, Wd), orc.expert_ffn(x, Wg, Wu, Wd2), atol=1e-13)
    assert not np.allclose(y0, orc.expert_ffn(x, Wg, Wu2, Wd))


def test_identical_experts_with_k_equal_n_reduce_to_one_dense_mlp():
    rng = np.random.default_rng(6)
    N, H, I, V = 3, 8, 10, 11
    w = _weights(rng, N, H, I, V)
    for name in ("w_gate", "w_up", "w_down"):
        w[name][:] = w[name][0]
    u = rng.standard_normal(H)
    x = orc.rmsnorm(u, None, 1e-5)
    s = orc.router_scores(x, w["router"])
    ids, g = orc.topk_gate(s, N)
    _, _, f = orc.moe_features(u, x, ids, g, w)
    dense = orc.expert_ffn(x, w["w_gate"][0], w["w_up"][0], w["w_down"][0])
    assert np.allclose(f - u, dense, atol=1e-12)       # sum_j s_j = 1


def test_branch_features_add_up_to_the_combined_feature():
    rng = np.random.default_rng(7)
    N, H, I, V = 4, 8, 6, 9
    w = _weights(rng, N, H, I, V)
    u = rng.standard_normal(H)
    x = orc.rmsnorm(u, None, 1e-5)
    ids, g = orc.topk_gate(orc.router_scores(x, w["router"]), 2)
    y, b, f = orc.moe_features(u, x, ids, g, w)
    assert np.allclose(b[0] + b[1] - u, f, atol=1e-12)
    # without the branch residual the branch is the literal s * Expert(x)
    y2, b2, f2 = orc.moe_features(u, x, ids, g, w, branch_residual=False)
    assert np.allclose(b2[0], g[0] * y[0]) and np.allclose(f2, f)
    # each branch uses its own expert only: changing the right expert leaves the left alone
    w2 = {k: v.copy() for k, v in w.items()}
    w2["w_down"][ids[1]] *= 2.0
    _, b3, _ = orc.moe_features(u, x, ids, g, w2)
    assert np.allclose(b3[0], b[0]) and not np.allclose(b3[1], b[1])


def test_coupled_degenerate_case_gives_identical_left_and_right_logits():
    rng = np.random.default_rng(8)
    N, H, I, V = 4, 8, 6, 13
    w = _weights(rng, N, H, I, V)
    for name in ("w_gate", "w_up", "w_down"):
        w[name][:] = w[name][0]
    w["router"][:] = w["router"][0]             # equal scores 1/N
    u = rng.standard_normal((1, 1, H))
    out = orc.draft_expand(u, np.zeros((1, 1)), w, k_e=3, width=4)
    assert np.allclose(out["gate"], 0.25)
    assert np.allclose(out["logits"][0, 0, 0], out["logits"][0, 0, 1], atol=1e-12)
    assert out["tok"][0, 0, 0].tolist() == out["tok"][0, 0, 1].tolist()


def test_head_is_a_plain_matrix_product():
    rng = np.random.default_rng(9)
    b = rng.standard_normal((2, 5))
    W = rng.standard_normal((7, 5))
    lg = orc.head_logits(b, W)
    for r in range(2):
        for v in range(7):
            assert lg[r, v] == pytest.approx(sum(b[r, k] * W[v, k] for k in range(5)), rel=1e-12)


# ----------------------------------------------------------------- per-expert top-k
def test_branch_topk_against_python_sort_and_normalisation():
    rng = np.random.default_rng(10)
    row = rng.standard_normal(37)
    row[5] = row[20] = row.max() + 1.0          # a tie for first place
    ids, score, lse = orc.branch_topk(row, 6, parent_score=-1.5)
    ref = sorted(range(37), key=lambda v: (-row[v], v))[:6]
    assert ids.tolist() == ref and ids[0] == 5 and ids[1] == 20
    z = sum(math.exp(t) for t in row)
    assert lse == pytest.approx(math.log(z), rel=1e-12)
    for j, v in enumerate(ref):
        assert score[j] == pytest.approx(-1.5 + math.log(math.exp(row[v]) / z), rel=1e-10)
    ids_all, score_all, _ = orc.branch_topk(row, 37, 0.0)
    assert np.exp(score_all).sum() == pytest.approx(1.0, rel=1e-12)
    assert np.all(np.diff(score_all) <= 0)


def test_frontier_select_order():
    sc = np.array([-3.0, -1.0, -2.0, -1.0, -5.0])
    assert orc.frontier_select(sc, 3).tolist() == [1, 3, 2]


# ----------------------------------------------------------------- tree growth
def _grow(seed, B=1, H=16, I=12, V=23, N=4, k_e=2, width=4, depth=4, same_u=False):
    rng = np.random.default_rng(seed)
    w = _weights(rng, N, H, I, V)
    fs = [1]
    for _ in range(1, depth):
        fs.append(min(width, fs[-1] * 2 * k_e))
    us = []
    for F in fs:
        if same_u:
            us.append(np.repeat(rng.standard_normal((B, 1, H)), F, axis=1))
        else:
            us.append(rng.standard_normal((B, F, H)))
    return w, fs, us, orc.grow_tree(us, w, k_e, width)


def test_unpruned_growth_is_the_full_product_tree():
    # width >= all candidates and the same u for every node of a layer: every node of a
    # layer has the same two child distributions, so the tree is a product structure
    k_e, depth = 2, 3
    w, fs, us, pool = _grow(11, k_e=k_e, width=1000, depth=depth, same_u=True)
    assert fs == [1, 4, 16]
    n = pool["tok"].shape[1]
    assert n == 4 + 16 + 64
    per_layer = []
    for l in range(depth):
        out = orc.draft_expand(us[l][:, :1], np.zeros((1, 1)), w, k_e, 1000)
        lp = out["score"][0, 0]                 # [K, k_e] log-probs (parent score 0)
        per_layer.append((out["tok"][0, 0], lp))
    # every root-to-node path = a sequence of (branch, rank) choices
    expect = {}
    for l in range(1, depth + 1):
        for choice in itertools.product(range(2 * k_e), repeat=l):
            sc = sum(per_layer[i][1].reshape(-1)[c] for i, c in enumerate(choice))
            toks = tuple(int(per_layer[i][0].reshape(-1)[c]) for i, c in enumerate(choice))
            expect[toks + (l,)] = expect.get(toks + (l,), []) + [sc]
    got = {}
    for g in range(n):
        toks = []
        t = g
        while t >= 0:
            toks.append(int(pool["tok"][0, t]))
            t = int(pool["parent"][0, t])
        key = tuple(reversed(toks)) + (len(toks),)
        got[key] = got.get(key, []) + [float(pool["score"][0, g])]
    assert set(got) == set(expect)
    for key in got:
        assert np.allclose(sorted(got[key]), sorted(expect[key]), atol=1e-10)


@pytest.mark.parametrize("seed", [12, 13, 14])
def test_pool_scores_are_path_sums_of_the_stored_distributions(seed):
    k_e = 2
    w, fs, us, pool = _grow(seed, k_e=k_e, width=4, depth=4)
    br = orc.pool_branches(fs, 2, k_e)
    n = pool["tok"].shape[1]
    assert n == sum(f * 2 * k_e for f in fs)
    for g in range(n):
        pg = int(pool["parent"][0, g])
        pslot = 0 if pg < 0 else int(pool["qslot"][0, pg])
        assert pslot >= 0                       # a node's parent was expanded
        row = pool["logits"][0, pslot, br[g]]
        logp = row[pool["tok"][0, g]] - math.log(np.exp(row).sum())
        base = 0.0 if pg < 0 else pool["score"][0, pg]
        assert pool["score"][0, g] == pytest.approx(base + logp, rel=1e-10, abs=1e-10)
    # expanded slots are 0..S-1, each used once
    used = sorted(int(s) for s in pool["qslot"][0] if s >= 0)
    assert used == list(range(1, sum(fs)))


@pytest.mark.parametrize("seed,M", [(15, 16), (16, 9), (17, 30)])
def test_final_tree_invariants(seed, M):
    k_e, D = 2, 4
    w, fs, us, pool = _grow(seed, k_e=k_e, width=4, depth=D)
    t = orc.tree_finalize(pool["tok"][0], pool["score"][0], pool["parent"][0], pool["qslot"][0],
                          root_tok=7, tree_size=M, frontier_sizes=fs, top_k=2, k_e=k_e)
    assert len(t["tok"]) == M and t["tok"][0] == 7 and t["parent"][0] == -1
    assert all(t["parent"][i] < i for i in range(1, M))
    assert np.all(np.diff(t["depth"]) >= 0) and t["depth"].max() <= D
    anc = orc.ancestor_mask(t["parent"])
    assert np.array_equal(anc.sum(1), t["depth"] + 1)
    # the kept set is the M-1 best of the pool: nothing left out scores above the worst kept
    kept = set(t["keep"].tolist())
    worst = min(pool["score"][0, g] for g in kept)
    for g in range(pool["tok"].shape[1]):
        if g not in kept:
            assert pool["score"][0, g] <= worst
    # children of one parent are contiguous and left-branch children come first
    for i in range(M):
        kids = orc.children_of(t["parent"], i)
        if kids:
            assert kids == list(range(kids[0], kids[0] + len(kids)))
            assert list(t["branch"][kids]) == sorted(t["branch"][kids])
    # scores never increase from parent to child
    for i in range(1, M):
        p = t["parent"][i]
        if p > 0:
            assert t["score"][i] <= t["score"][p] + 1e-12


def test_tree_finalize_rejects_a_pool_that_is_too_small():
    with pytest.raises(ValueError):
        orc.tree_finalize(np.zeros(3, np.int32), np.zeros(3), np.full(3, -1), np.full(3, -1),
                          0, 6, pool_branch=np.zeros(3, np.int32))
